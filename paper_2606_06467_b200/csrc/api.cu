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
        cudaDeviceGetAttribute(&d.l2_bytes, cudaDevAttrL2CacheSize, dev) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    cache[dev] = d;
    have[dev] = true;
  }
  *out = cache[dev];
  return true;
}

WorkspaceLayout make_workspace_layout(const clsa_params& p, const DeviceInfo& dev) {
  (void)dev;
  WorkspaceLayout w;
  auto align = [](size_t x) { return (x + 255) / 256 * 256; };
  w.scores_off = kStatusBytes;
  w.score_stride = ((int64_t)p.max_seq_len + 63) / 64 * 64;
  w.scores_bytes = align((size_t)p.num_seqs * p.q_per_seq * w.score_stride * sizeof(float));
  w.total = w.scores_off + w.scores_bytes;
  return w;
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
  if (p->sweep != 0 && p->sweep != 1) return CLSA_ERR_INVALID_ARG;
  if (p->attn_plan < 0 || p->attn_plan > 2) return CLSA_ERR_INVALID_ARG;
  if (p->max_seq_len < p->q_per_seq) return CLSA_ERR_INVALID_ARG;
  if (!isfinite(p->sm_scale) || !(p->sm_scale > 0.f)) return CLSA_ERR_INVALID_ARG;  // the kernels take maxima before scaling
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

#define CLSA_TRY(expr)                     \
  do {                                     \
    const clsa_status st__ = (expr);       \
    if (st__ != CLSA_OK) return st__;      \
  } while (0)

clsa_status from_cuda(cudaError_t e) { return e == cudaSuccess ? CLSA_OK : CLSA_ERR_CUDA; }

// The L attention launches that share one index. Layer 0 follows whatever produced the index and must wait for it;
// every later layer reads only what was complete before its predecessor started (the index, the caches, the caller's
// queries), so it does not wait, and several layers are in flight at once. All of them walk the selected set in the
// same direction (p.sweep): a layer then trails its predecessor by a few microseconds over the same rows and finds
// them in L2 (measured at the headline: 286 us per step against 320 us with alternating directions).
cudaError_t launch_layers(const clsa_params& p, const void* const* q_layers, void* const* out_layers, const int32_t* idx,
                          const int32_t* count, uint32_t* status, const DeviceInfo& dev, cudaStream_t s) {
  const ChainTail tail = chain_fine_tail(p, dev);  // the end of the chain uses smaller blocks so that it ends flush
  for (int l = 0; l < p.num_layers; ++l) {
    const bool fine = l >= p.num_layers - tail.layers;
    const int fine_rows = l == p.num_layers - tail.layers - 1 ? tail.rows : 0;  // the layer where the finer shape begins
    const cudaError_t err = launch_sparse_attn(p, q_layers[l], idx, count, out_layers[l], nullptr, status, p.sweep & 1,
                                               l == 0 ? 1 : 0, l + 1 < p.num_layers ? 1 : 0, fine ? 2 : 1, fine_rows, dev, s);
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

clsa_status clsa_sparse_attn(const clsa_params* p, const void* q, const int32_t* idx, const int32_t* count, void* out,
                             float* lse, void* workspace, size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_kv_cache(p));
  if (q == nullptr || idx == nullptr || count == nullptr || out == nullptr) return CLSA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(out, 16) || !aligned(idx, 4) || !aligned(count, 4) || !aligned(lse, 4))
    return CLSA_ERR_INVALID_ARG;
  CLSA_TRY(check_workspace(workspace, workspace_bytes, kStatusBytes));
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  return from_cuda(launch_sparse_attn(*p, q, idx, count, out, lse, static_cast<uint32_t*>(workspace), p->sweep & 1, 1, 0,
                                      p->attn_plan, 0, dev,
                                      static_cast<cudaStream_t>(stream)));
}

clsa_status clsa_decode_step(const clsa_params* p, const void* q_idx, const void* const* q_layers,
                             void* const* out_layers, int32_t* idx, int32_t* count, void* workspace,
                             size_t workspace_bytes, clsa_stream stream) {
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
  if (workspace == nullptr || !aligned(workspace, 256)) return CLSA_ERR_WORKSPACE;
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  const WorkspaceLayout w = make_workspace_layout(*p, dev);
  CLSA_TRY(check_workspace(workspace, workspace_bytes, w.total));
  auto base = static_cast<unsigned char*>(workspace);
  auto status = reinterpret_cast<uint32_t*>(base);
  auto scores = reinterpret_cast<float*>(base + w.scores_off);
  auto s = static_cast<cudaStream_t>(stream);
  cudaError_t err = launch_index_scores_decode(*p, q_idx, scores, w.score_stride, status, status + kSchedWord, dev, s);
  if (err != cudaSuccess) return CLSA_ERR_CUDA;
  err = launch_topk(*p, scores, w.score_stride, idx, count, status, dev, s);
  if (err != cudaSuccess) return CLSA_ERR_CUDA;
  if (launch_layers(*p, q_layers, out_layers, idx, count, status, dev, s) != cudaSuccess) return CLSA_ERR_CUDA;
  return CLSA_OK;
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
  CLSA_TRY(check_workspace(workspace, workspace_bytes, kStatusBytes));
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  return from_cuda(launch_layers(*p, q_layers, out_layers, idx, count, static_cast<uint32_t*>(workspace), dev,
                                 static_cast<cudaStream_t>(stream)));
}

clsa_status clsa_project_append(const clsa_params* p, int32_t d_model, const void* h, const void* w_q_idx,
                                const void* w_k_idx, const void* w_k, const void* w_v, void* q_idx_out,
                                void* workspace, size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_idx_cache(p));
  if (h == nullptr || w_q_idx == nullptr || w_k_idx == nullptr || q_idx_out == nullptr) return CLSA_ERR_INVALID_ARG;
  if ((w_k == nullptr) != (w_v == nullptr)) return CLSA_ERR_INVALID_ARG;
  if (!aligned(h, 16) || !aligned(w_q_idx, 16) || !aligned(w_k_idx, 16) || !aligned(w_k, 16) || !aligned(w_v, 16) ||
      !aligned(q_idx_out, 16))
    return CLSA_ERR_INVALID_ARG;
  if (d_model < 32) return CLSA_ERR_INVALID_ARG;
  if (d_model % 32 != 0) return CLSA_ERR_UNSUPPORTED;
  if (w_k != nullptr) CLSA_TRY(check_kv_cache(p));
  CLSA_TRY(check_workspace(workspace, workspace_bytes, kStatusBytes));
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  return from_cuda(launch_project_append(*p, d_model, h, w_q_idx, w_k_idx, w_k, w_v, q_idx_out,
                                         static_cast<uint32_t*>(workspace), dev, static_cast<cudaStream_t>(stream)));
}

// ---- entry point that allocates nothing -----------------------------------------------------------
// Scratch of clsa_decode_step_static: the status word followed by the fp32 score matrix, in a
// file-scope device array that every GPU loading this library keeps until the process exits.
namespace {
constexpr size_t kStaticScoreSlots = (size_t)2 << 20;  // 2 Mi fp32 scores = 8 MiB
constexpr size_t kStaticScratchBytes = kStatusBytes + kStaticScoreSlots * sizeof(float);
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
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_idx_cache(p));
  CLSA_TRY(check_kv_cache(p));
  if (q_idx == nullptr || q_layers == nullptr || out_layers == nullptr || idx == nullptr || count == nullptr)
    return CLSA_ERR_INVALID_ARG;
  if (!aligned(q_idx, 16) || !aligned(idx, 4) || !aligned(count, 4) || !aligned(dev_status, 4)) return CLSA_ERR_INVALID_ARG;
  for (int l = 0; l < p->num_layers; ++l)
    if (q_layers[l] == nullptr || out_layers[l] == nullptr || !aligned(q_layers[l], 16) || !aligned(out_layers[l], 16))
      return CLSA_ERR_INVALID_ARG;
  if (p->q_per_seq != 1) return CLSA_ERR_UNSUPPORTED;
  const int64_t stride = ((int64_t)p->max_seq_len + 63) / 64 * 64;
  if ((uint64_t)p->num_seqs * (uint64_t)stride > kStaticScoreSlots) return CLSA_ERR_WORKSPACE;  // beyond the fixed scratch
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  unsigned char* base = nullptr;
  if (static_scratch_address(&base) != cudaSuccess) return CLSA_ERR_CUDA;
  auto s = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left: the status word must start at zero. The score
  // matrix needs no clearing (every entry that is read is written first).
  uint32_t* status = dev_status != nullptr ? dev_status : reinterpret_cast<uint32_t*>(base);
  if (dev_status == nullptr && cudaMemsetAsync(base, 0, kStatusBytes, s) != cudaSuccess) return CLSA_ERR_CUDA;
  auto scores = reinterpret_cast<float*>(base + kStatusBytes);
  // the score kernel's scheduling counters always live in the scratch array's header (zero when the library is
  // loaded, and left at zero by every launch), also when the status word is the caller's
  if (launch_index_scores_decode(*p, q_idx, scores, stride, status, reinterpret_cast<uint32_t*>(base) + kSchedWord, dev, s) !=
      cudaSuccess)
    return CLSA_ERR_CUDA;
  if (launch_topk(*p, scores, stride, idx, count, status, dev, s) != cudaSuccess) return CLSA_ERR_CUDA;
  if (launch_layers(*p, q_layers, out_layers, idx, count, status, dev, s) != cudaSuccess) return CLSA_ERR_CUDA;
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

int clsa_version(void) { return 100; }

}  // extern "C"
