/*
 * clsa.h -- C ABI of the CLSA decoding hot path for NVIDIA B200 (sm_100a).
 *
 * Cross-layer sparse attention shares one routing index between all cross-decoder layers that read
 * the same KV cache. The path behind this boundary is the part of a decode (or prefill-chunk) step
 * that touches the caches:
 *
 *   1. index scores   I = Q_idx K_idx^T                      (Eq. 3; single indexer head, Eq. 2)
 *   2. routing index  S_t = TopK(I_t, k), once per query     (Eq. 3)
 *   3. per layer l    O_t^(l) = Attn(Q_t^(l), K_{S_t}, V_{S_t}) (Eq. 4), every layer reusing S_t
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 * Pointers: every pointer is a DEVICE pointer unless its comment says HOST. The clsa_params struct
 *   itself lives in host memory and is read during the call only. "Device pointer" means any address
 *   the device can dereference: the attention outputs, which are written once with plain stores, may
 *   for example live in pinned host memory mapped into the unified address space (a decode step's
 *   outputs then reach the host without a copy). Inputs that many blocks read (q_idx, the caches, the
 *   index) belong in device memory: the kernels' traffic assumptions hold only there.
 * Ownership: the caller owns every buffer (inputs, outputs, workspace). The library allocates
 *   nothing, frees nothing, keeps no state between calls except cached device properties, and only
 *   enqueues work on the given stream. No entry point synchronises except clsa_device_status.
 * Errors: each call returns a clsa_status. All argument checks run on the host before anything is
 *   enqueued: a call that returns CLSA_ERR_INVALID_ARG, CLSA_ERR_UNSUPPORTED or CLSA_ERR_WORKSPACE
 *   has launched nothing. Unsupported shapes are refused, never routed to a slower path.
 *   Data-dependent problems seen on the device (an index outside its sequence, a sequence longer
 *   than max_seq_len) never trap: the offending element is skipped and a bit is set in the status
 *   word at the start of the workspace (see clsa_device_status).
 * Layout: bf16 = IEEE bfloat16 bit patterns. Strides are in elements. Cache rows of sequence b are
 *   rows seq_start[b] .. seq_start[b] + seq_len[b] - 1 of one row space shared by K, V and K_idx (or, with a
 *   block table, the rows of its blocks: see clsa_params).
 *   The last q_per_seq tokens of a sequence are its query tokens (their own K/V/K_idx rows have
 *   already been appended by the caller).
 * Visibility: with causal == 0 every query sees all seq_len[b] tokens (decoding); with causal == 1
 *   query t (0-based, of T = q_per_seq) sees positions s <= seq_len[b] - T + t.
 * Index contract: idx holds, per (sequence, query), `count` distinct sequence-local positions in
 *   [0, visible); entries at or beyond count are -1. clsa_topk emits them in ascending position
 *   order; clsa_sparse_attn accepts any order.
 */
#ifndef CLSA_H_
#define CLSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define CLSA_API __attribute__((visibility("default")))
#else
#define CLSA_API
#endif

typedef enum {
  CLSA_OK = 0,
  CLSA_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, misaligned pointer or stride */
  CLSA_ERR_UNSUPPORTED = 2, /* valid but not built: head_dim != 128, idx_dim not in {64,128}, group size > 16 ... */
  CLSA_ERR_WORKSPACE = 3,   /* workspace null, misaligned (256 B) or smaller than clsa_workspace_bytes */
  CLSA_ERR_CUDA = 4         /* a CUDA runtime call or launch failed; cudaGetLastError has the detail */
} clsa_status;

/* Bits of the device status word (first 4 bytes of the workspace, cleared by the host of the caller
 * or by clsa_clear_status; kernels only ever OR into it). */
#define CLSA_DEV_BAD_INDEX 1u   /* an idx entry < 0 or >= seq_len inside the first `count` entries: skipped */
#define CLSA_DEV_BAD_SEQLEN 2u  /* seq_len[b] < q_per_seq or > max_seq_len: that sequence was skipped */
#define CLSA_DEV_BAD_COUNT 4u   /* count[b,t] < 0 or > top_k: clamped */
#define CLSA_DEV_TIMEOUT 8u     /* a bounded wait inside a kernel ran out; the kernel returned early, results are invalid */
#define CLSA_DEV_BAD_WORKSPACE 16u /* the workspace header was not zero before its first use (the score kernel found its
                                      scheduling counters out of range): results are invalid */

#define CLSA_DEV_ROUTING_OVERFLOW 32u /* clsa_index_topk: more rows than its scratch holds had to be recomputed from the
                                        full score row (long runs of equal scores, non-finite scores); the surplus rows
                                        have count 0: route them with clsa_index_scores + clsa_topk */

typedef void* clsa_stream; /* a cudaStream_t */

typedef struct {
  int32_t num_seqs;     /* B >= 1 */
  int32_t q_per_seq;    /* T >= 1: 1 = decode; > 1 = prefill chunk */
  int32_t num_q_heads;  /* Hq; Hq % Hkv == 0; group size Hq/Hkv <= 16 */
  int32_t num_kv_heads; /* Hkv */
  int32_t head_dim;     /* D == 128 */
  int32_t idx_dim;      /* d_idx: 64 or 128 */
  int32_t top_k;        /* k >= 1: the maximum number of activated tokens per query */
  int32_t num_layers;   /* L >= 1; read by clsa_decode_step and clsa_workspace_bytes only */
  int32_t causal;       /* 0 or 1, see "Visibility" */
  int32_t max_seq_len;  /* host-known upper bound of seq_len[], used for grid sizing (no device read-back) */
  float sm_scale;       /* softmax scale of Eq. 4's Attn; finite and > 0 (the kernels take running maxima over the raw
                           dot products, which is only valid for a positive scale; other values are refused with
                           CLSA_ERR_INVALID_ARG); 1/sqrt(head_dim) in the benchmarks */
  const int64_t* seq_start; /* [B] first cache row of each sequence */
  const int32_t* seq_len;   /* [B] valid tokens n_b >= T, including the T query tokens */
  const void* k_cache;      /* bf16 [rows][Hkv][D]; element (r,g,d) at r*kv_token_stride + g*kv_head_stride + d */
  const void* v_cache;      /* bf16, same layout and strides as k_cache */
  int64_t kv_token_stride;  /* multiple of 8 (16-byte rows) */
  int64_t kv_head_stride;   /* multiple of 8 */
  const void* idx_k_cache;  /* bf16 [rows][d_idx]; element (r,j) at r*idx_token_stride + j */
  int64_t idx_token_stride; /* multiple of 8 */
  int64_t num_cache_rows;   /* rows of the cache row space (the extent of k_cache, v_cache and idx_k_cache); required when
                               q_per_seq > 1, where tiled bulk copies need the bound. Optional (0 = unknown) otherwise; when
                               given, clsa_sparse_attn computes row addresses in 32 bits where the caches allow it and treats
                               a row at or beyond the extent like an index outside its sequence (skipped and flagged) */
  /* Paged caches (optional). With block_table == NULL sequence b occupies the contiguous rows starting at
   * seq_start[b]. Otherwise the row space is cut into blocks of block_size rows and position s of sequence b is
   * cache row  block_table[b * max_blocks_per_seq + s / block_size] * block_size + s % block_size  (the same
   * mapping for K, V and K_idx); seq_start is then ignored and may be NULL. */
  const int32_t* block_table; /* int32 [B][max_blocks_per_seq] physical block numbers, or NULL */
  int32_t block_size;         /* a power of two, 16 .. 4096 (paged only) */
  int32_t max_blocks_per_seq; /* >= ceil(max_seq_len / block_size) (paged only) */
} clsa_params;

/* Bytes of workspace that any of the calls below may need for these params (the maximum over them:
 * the status header, the scratch through which a standalone decode clsa_sparse_attn merges the
 * partial results of its blocks -- arrival counters and partial slots -- and the fp32 score matrix
 * that clsa_decode_step keeps there). Reads only the scalar fields. *bytes is HOST memory. The workspace must be 256-byte aligned
 * and ALL of it zero before the first call (cudaMemset): its first 256 bytes hold the device status
 * word and the score kernel's scheduling counters, the attention scratch begins with arrival counters;
 * every launch leaves all of these counters at zero again, and clsa_clear_status zeroes the status word.
 * Calls that overlap on the GPU must not share a workspace. */
CLSA_API clsa_status clsa_workspace_bytes(const clsa_params* p, size_t* bytes);

/* Eq. 3, first half: scores[b][t][s] = sum_j q_idx[b][t][j] * K_idx[seq_start[b]+s][j] for every
 * visible s; the bare dot product, no scale and no activation, one indexer head. bf16 products are
 * exact in fp32; accumulation is fp32. Entries at s >= visible(b,t) are not written.
 *   q_idx  bf16 [B][T][d_idx], 16-byte aligned
 *   scores fp32 [B][T][score_stride], score_stride >= max_seq_len
 * T == 1 streams the indexer-key cache once (HBM-bound); T > 1 is a tensor-core GEMM (tcgen05, operands staged by
 * TMA), which needs p->num_cache_rows and, for 32-byte vector stores, a 32-byte aligned `scores` with
 * score_stride % 8 == 0 (otherwise it falls back to scalar stores of the same values). Both paths accept paged
 * caches (T > 1 fetches one tiled copy per cache block; num_cache_rows is then the extent of the paged row space). */
CLSA_API clsa_status clsa_index_scores(const clsa_params* p, const void* q_idx, float* scores, int64_t score_stride,
                              void* workspace, size_t workspace_bytes, clsa_stream stream);

/* Eq. 3, second half: per (b,t) the c = min(k, visible) positions with the largest scores, ties to
 * the lower position, -0.0 equal to +0.0. Fewer than k visible tokens selects all of them (k is a
 * maximum). Exact selection: no approximation, no sampling.
 *   idx   int32 [B][T][k]  ascending positions, tail -1
 *   count int32 [B][T]
 * Scores must be finite; a NaN is ordered by its bit pattern and never faults. */
CLSA_API clsa_status clsa_topk(const clsa_params* p, const float* scores, int64_t score_stride, int32_t* idx,
                      int32_t* count, void* workspace, size_t workspace_bytes, clsa_stream stream);

/* Eq. 3 in one call: S = TopK(Q_idx K_idx^T, k) per (b,t), the same idx and count as clsa_index_scores followed by
 * clsa_topk, bit for bit. For a prefill chunk (T > 1) the T x n score matrix is never written to memory: the
 * contraction runs on the tensor cores once over a sample of the keys, which gives every query row a pivot safely
 * below its k-th largest score, and once over all keys with an epilogue that keeps only the scores not below the
 * pivot as (score, position) candidates; an exact selection over the candidates gives the index. Rows whose
 * candidates cannot give the exact answer (long runs of equal scores at the threshold, non-finite scores) are
 * recomputed through a small scratch matrix; if more than 64 rows of one call need that, the surplus rows get
 * count 0 and CLSA_DEV_ROUTING_OVERFLOW is set (see there). Shapes the fused route does not take (k so large, or rows
 * so long, that its fixed-size lists or bitmaps would not hold them) and T == 1 run the two calls internally, with
 * the scores in the workspace.
 *   q_idx bf16 [B][T][d_idx], 16-byte aligned;  idx int32 [B][T][k], count int32 [B][T] as for clsa_topk
 * Needs p->num_cache_rows when T > 1 and the whole workspace of clsa_workspace_bytes. */
CLSA_API clsa_status clsa_index_topk(const clsa_params* p, const void* q_idx, int32_t* idx, int32_t* count, void* workspace,
                                     size_t workspace_bytes, clsa_stream stream);

/* Eq. 4 for ONE layer: for each (b,t) and query head h with KV head g = h / (Hq/Hkv),
 *   O = sum_{s in S} softmax_s(sm_scale * Q[b][t][h] . K[s][g]) V[s][g]   over the selected rows only.
 * No positional rotation is applied (the cross-decoder's global attention is NoPE). p->sm_scale must be finite and
 * greater than zero (CLSA_ERR_INVALID_ARG otherwise): a restriction of this library, not of Eq. 4 -- the kernels take
 * running maxima over the raw dot products and apply the scale afterwards.
 *   q   bf16 [B][T][Hq][D]           this layer's queries, 16-byte aligned
 *   out bf16 [B][T][Hq][D]           round-to-nearest-even from fp32 accumulators
 *   lse fp32 [B][T][Hq] or NULL      log-sum-exp of the scaled logits (natural log)
 * A (b,t) with count 0 yields zeros and lse = -inf. A sequence with seq_len < T or > max_seq_len is treated as
 * count 0 and flags CLSA_DEV_BAD_SEQLEN (its index entries are never used as addresses).
 * The launch assumes nothing about what runs before it on the stream and waits for it; it has the whole GPU to
 * itself (the shape for a layer whose output feeds the next kernel). Needs the whole workspace of
 * clsa_workspace_bytes when T == 1 (such launches merge the partial results of their blocks through it). */
CLSA_API clsa_status clsa_sparse_attn(const clsa_params* p, const void* q, const int32_t* idx, const int32_t* count,
                             void* out, float* lse, void* workspace, size_t workspace_bytes, clsa_stream stream);

/* What a caller knows about the launches around one clsa_sparse_attn call. Hints select the launch shape and the
 * order of memory accesses; they never change what is computed (results of different hints agree to rounding: the
 * selected set is split differently), and all-zero hints are always valid. */
typedef struct {
  int32_t reverse;        /* 0 or 1: walk the selected set from its end. A decoder that issues its layers one by one
                             alternates this from layer to layer, so that a layer starts on the rows its predecessor
                             fetched last (still in L2). */
  int32_t shared_gpu;     /* 0: the launch has the GPU to itself (the work is cut at token granularity over all SMs).
                             1: it runs side by side with its neighbours on the stream (launches that do not wait for
                             one another, as the L layers of clsa_decode_step): a few large blocks, about 32 per launch.
                             2: as 1 with half the KV heads per block where that is possible (twice the blocks); the
                             chained calls use it for their last layers so that the chain's blocks keep every SM
                             busy to the end (see clsa_chain_plan).
                             3: the block shape of the launches in which the chained calls compute two layers at once
                             (see clsa_chain_plan), for one layer: a few larger blocks, about 16 per launch; which
                             shape that is depends on p->num_layers too (how many such launches share the GPU).
                             4: as 3 with half the KV heads per block where the chain's plan allows it; the chained
                             calls use it for their last pairs of layers. */
  int32_t keep_rows;      /* 1: another launch that reads the same selected rows follows (the next layer): fetch them
                             with the L2 evict_last priority so that other traffic does not push them out in between. */
  int32_t only_q_pending; /* 1: idx, count, seq_len, the block table and the caches were all complete before the kernel
                             in front of this call on the stream was launched; only q may still be in the making
                             (every layer of a decoder after the first). The row copies then start before the launch
                             waits for that kernel. Setting it when the index is still being written reads a stale
                             index. */
} clsa_attn_hints;

/* clsa_sparse_attn with hints (NULL = all zero = clsa_sparse_attn). */
CLSA_API clsa_status clsa_sparse_attn_hinted(const clsa_params* p, const void* q, const int32_t* idx, const int32_t* count,
                                    void* out, float* lse, const clsa_attn_hints* hints, void* workspace,
                                    size_t workspace_bytes, clsa_stream stream);

/* One step (Sec. 2.1: the routing index is computed once and shared by the layers): index scores, TopK, then L
 * sparse-attention launches on `stream`, all fed the same idx/count, which are returned.
 *   q_layers   HOST array of L device pointers, each bf16 [B][T][Hq][D]
 *   out_layers HOST array of L device pointers, each bf16 [B][T][Hq][D]
 * Equivalent, bit for bit, to clsa_index_scores, clsa_topk and L calls of clsa_sparse_attn_hinted made one after
 * another with hints {reverse 0, shared_gpu 3 (or 4) for the layers that clsa_chain_plan reports as computed two per
 * launch (in the finer shape), else 1 (or 2), keep_rows 1 except for the last layer}. Two layers per launch (decoding, groups of
 * up to 8 query heads per KV head): every layer gathers the same rows, so a launch that has two layers' queries copies
 * the rows from L2 once for both. The layers do not wait for one another (each reads only the index, the caches and its own queries, all of which the caller
 * hands over up front), so several of them are in flight at once and share the selected rows through L2. A decoder
 * whose layer l+1 queries depend on layer l's output cannot use this call: it issues clsa_index_scores, clsa_topk
 * and one clsa_sparse_attn_hinted per layer instead. T > 1 is not chained here. */
CLSA_API clsa_status clsa_decode_step(const clsa_params* p, const void* q_idx, const void* const* q_layers,
                             void* const* out_layers, int32_t* idx, int32_t* count, void* workspace,
                             size_t workspace_bytes, clsa_stream stream);

/* Eq. 4 for all L layers that share one index (Sec. 2.1): the attention half of clsa_decode_step on its own, for a
 * caller that has the index already (from clsa_index_scores + clsa_topk) -- for instance to let the layers' queries
 * arrive on another stream while the routing runs, making `stream` wait on that upload just before this call.
 *   q_layers / out_layers  HOST arrays of L device pointers, each bf16 [B][T][Hq][D], 16-byte aligned
 *   idx, count             as written by clsa_topk (read only)
 * Bit for bit the L calls of clsa_sparse_attn_hinted with the hints given under clsa_decode_step and lse = NULL,
 * launched so that a layer does not wait for its predecessor (which is why the calls are offered as one). */
CLSA_API clsa_status clsa_sparse_attn_layers(const clsa_params* p, const void* const* q_layers, const int32_t* idx,
                                             const int32_t* count, void* const* out_layers, void* workspace,
                                             size_t workspace_bytes, clsa_stream stream);

/* The step immediately before the path (Eq. 2 and the append of the new tokens' cache rows): for query token t
 * of sequence b, at position s = seq_len[b] - T + t (the sequence's newest tokens, whose rows this call fills),
 *   q_idx_out[b][t][:]        = h[b][t][:] W^Q_idx                     (Eq. 2)
 *   K_idx cache row of (b,s)  = h[b][t][:] W^K_idx                     (Eq. 2)
 *   K and V cache rows of (b,s), laid out [Hkv][D] = h W^K, h W^V      (the shared cache built from the same states)
 * bf16 operands, fp32 accumulation, one round-to-nearest-even to bf16. No normalisation, bias or rotation.
 *   d_model  hidden size, a multiple of 32 (otherwise CLSA_ERR_UNSUPPORTED)
 *   h        bf16 [B][T][d_model], 16-byte aligned
 *   w_q_idx, w_k_idx  bf16 [d_idx][d_model]: one OUTPUT feature per row (y[o] = sum_j h[j] * w[o][j]), 16-byte aligned
 *   w_k, w_v bf16 [Hkv*D][d_model], feature g*D + d is element d of KV head g; both NULL = indexer branch only
 *   q_idx_out bf16 [B][T][d_idx], 16-byte aligned
 *   idx_k_cache_out          the K_idx cache, writable: same address, layout and paging as p->idx_k_cache describes
 *   k_cache_out, v_cache_out the K and V caches, writable (both NULL together with w_k and w_v)
 * The call writes exactly the cache rows above through these three pointers and nothing else; p's own (const) cache
 * pointers are not written through and need not be set. seq_len must already count the new tokens. Calls that
 * follow on the same stream (clsa_index_scores, clsa_decode_step) see the appended rows. A sequence with
 * seq_len < T or > max_seq_len is skipped and flags CLSA_DEV_BAD_SEQLEN. Built for decoding (B*T up to a few
 * dozen rows, where the op is a stream of the weights); larger B*T works but re-reads the weights per 64 rows. */
CLSA_API clsa_status clsa_project_append(const clsa_params* p, int32_t d_model, const void* h, const void* w_q_idx,
                                         const void* w_k_idx, const void* w_k, const void* w_v, void* q_idx_out,
                                         void* idx_k_cache_out, void* k_cache_out, void* v_cache_out,
                                         void* workspace, size_t workspace_bytes, clsa_stream stream);

/* The same step as clsa_decode_step for callers that cannot allocate device memory. (The paper has
 * no counterpart: this is a convenience of the library.) Some callers have no way to obtain a
 * workspace: code that runs inside a region where cudaMalloc is forbidden or would synchronise the
 * device (a latency-critical serving loop, a plug-in that is handed tensors but no allocator, a
 * process whose memory pool is already fully reserved). For them the scratch that clsa_decode_step
 * keeps in the caller's workspace -- the status header and the fp32 score matrix (the chained
 * attention launches need none of the scratch that a standalone clsa_sparse_attn does) -- lives in a
 * device array built into the library: 16 MiB + 256 bytes per GPU that loads the library, held until
 * the process exits. This entry point calls no cudaMalloc, cudaFree or any other allocating routine.
 *   Limit: clsa_workspace_bytes(p) <= 16 MiB + 256 bytes (for example 16 sequences of 131 072 tokens
 *     with 32/8 heads: 8 MiB of scores behind 4.3 MiB of attention scratch that this entry point
 *     leaves unused); larger shapes return CLSA_ERR_WORKSPACE and launch nothing. T must be 1.
 *   dev_status: DEVICE pointer to one uint32 owned by the caller that receives the CLSA_DEV_* bits
 *     (the caller zeroes it), or NULL to drop them into the built-in array's own word.
 *   First call on a device: looks up the array's device address (once per device, with that device
 *     current). Make this first call outside any stream capture.
 *   Sharing: every call on a GPU uses the same array, which still holds the previous call's
 *     contents. Every call begins by zeroing the array's header (status word and scheduling
 *     counters) on `stream`, so a call that was cut short (or two calls that raced) cannot poison
 *     later ones; the scores need no clearing (every entry that is read is written first). Two calls whose GPU work overlaps
 *     (different streams, or different threads) race on the array and give wrong results for those
 *     calls. Serialise them, or use clsa_decode_step with one workspace per stream.
 * All other arguments, results and error behaviour are those of clsa_decode_step, with which the
 * results agree bit for bit. */
CLSA_API clsa_status clsa_decode_step_static(const clsa_params* p, const void* q_idx, const void* const* q_layers,
                                             void* const* out_layers, int32_t* idx, int32_t* count,
                                             uint32_t* dev_status, clsa_stream stream);

/* Measurement aid (the paper has no counterpart): the memory accesses of one decode clsa_sparse_attn launch -- the
 * same split of the selected set over the SMs, the same 16-byte asynchronous copies of K and V rows into the same
 * shared-memory ring -- with the arithmetic, the queries and the outputs left out. Timing it on rows that are, or
 * are not, resident in L2 gives the rate the memory system delivers to this access pattern, the ceiling that the
 * attention kernel is measured against. T must be 1. hints as for clsa_sparse_attn_hinted (NULL = all zero;
 * shared_gpu and only_q_pending are ignored: the probe is the shape of a launch that has the GPU to itself). Writes
 * only into the workspace (which must be the whole clsa_workspace_bytes). It leaves its own device-side duration in
 * the workspace header, free of launch overheads: bytes 8..15 hold the bitwise complement of the earliest start of
 * any of its warps and bytes 16..23 the latest end, both uint64 nanoseconds of the GPU's global timer; both words
 * accumulate by maximum, so clear the header (clsa_clear_status) before a launch that is to be read. */
CLSA_API clsa_status clsa_gather_probe(const clsa_params* p, const int32_t* idx, const int32_t* count,
                                       const clsa_attn_hints* hints, void* workspace, size_t workspace_bytes,
                                       clsa_stream stream);

/* Host only, no CUDA call: the launch shapes of an L-layer chain (clsa_decode_step, clsa_sparse_attn_layers) on a device
 * with `sm_count` SMs and a peak SM clock of `clock_khz`. The first *paired_layers layers (an even number) are computed
 * two per launch (groups of up to 8 query heads: all but an odd last layer), the last *fine_layers of them in the finer
 * shape (shared_gpu = 4), the rest in shape 3. With *paired_layers = 0 (wider groups) the last *fine_layers layers use
 * the finer one-layer shape (shared_gpu = 2), the rest shape 1. *fine_layers = 0: one shape throughout; always so for
 * T > 1 and for devices the block model was not measured on. The finer tail comes from a model of how the chain's blocks
 * fill the SMs; it costs a few microseconds the first time a shape is seen and is remembered afterwards. Outputs are
 * HOST pointers. */
CLSA_API clsa_status clsa_chain_plan(const clsa_params* p, int32_t sm_count, int32_t clock_khz, int32_t* fine_layers,
                                     int32_t* paired_layers);

/* Zero the status word (asynchronous, on `stream`). */
CLSA_API clsa_status clsa_clear_status(void* workspace, size_t workspace_bytes, clsa_stream stream);

/* Copy the device status word to *bits (HOST). Synchronises `stream`. */
CLSA_API clsa_status clsa_device_status(const void* workspace, uint32_t* bits, clsa_stream stream);

/* Static string for a status code. */
CLSA_API const char* clsa_status_string(clsa_status s);

/* Library version: major * 10000 + minor * 100 + patch. */
CLSA_API int clsa_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CLSA_H_ */
