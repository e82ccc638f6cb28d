/* jupiter.h — C ABI of the B200 (sm_100a) KV-cache attention library.
 *
 * The library implements the one data-parallel hot path behind the two
 * contributions of "Jupiter" (arXiv 2504.08242): attention of a query block
 * against a growing KV cache.
 *
 *   - Sec. II-A: a decoder layer's masked multi-head attention reads the keys
 *     and values of all previous tokens from the KVCache.
 *   - Sec. IV-A ("Opportunities of Intra-Sequence Parallel Inference",
 *     Fig. 5(b)): a prompt is cut into sub-sequences; sub-sequence s_i attends
 *     to the cached states of s_1..s_{i-1} plus its own causal block.
 *   - Sec. V-A (Fig. 7, steps 3 and 5): k candidate tokens are verified in one
 *     pass with their K/V stored in the cache; rejected ones are removed.
 *   - Sec. V-B (Fig. 8): all point-extending requests share the prompt's
 *     KVCache.
 *
 * Conventions shared by every call
 *   - All tensor pointers are DEVICE pointers unless a parameter says "host".
 *     They are caller-owned and only borrowed until the enqueued work ends.
 *   - bf16 inputs, fp32 outputs, fp32 accumulation.
 *   - Token-major tensors (q, k_new, v_new, out) are dense [batch][rows][heads][D].
 *   - A cache is head-major: element (b, h, row, d) of k or v lives at
 *     b*stride_batch + h*stride_head + row*stride_row + d (in elements);
 *     D contiguous, stride_row >= D, every stride a multiple of 8 elements and
 *     both base pointers 16-byte aligned.
 *   - Grouped-query attention: query head h reads KV head h / (q_heads/kv_heads).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*,
 *     NULL = default stream).  Every argument error is found on the host before
 *     anything is enqueued; outputs are then untouched and the status says why.
 *   - A ctx is bound to one device and must be used by one host thread and one
 *     stream at a time (its split-KV scratch is shared by successive calls in
 *     stream order).
 *   - Supported: head_dim 64 or 128; q_heads a multiple of kv_heads; any
 *     pos >= 0 and q_len >= 1 (no tile-multiple requirement).
 */
#ifndef JUPITER_H_
#define JUPITER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct jupiter_ctx jupiter_ctx;

typedef enum {
  JUPITER_OK = 0,
  JUPITER_ERR_INVALID_ARG = 1,  /* NULL pointer, non-positive size, bad head counts */
  JUPITER_ERR_OUT_OF_RANGE = 2, /* pos + rows beyond capacity, length beyond capacity */
  JUPITER_ERR_UNSUPPORTED = 3,  /* head_dim not 64/128, q_len too large for the branch path, device not sm_100 */
  JUPITER_ERR_ALIGNMENT = 4,    /* pointer or stride not 16-byte aligned */
  JUPITER_ERR_WORKSPACE = 5,    /* the ctx scratch is too small for this call */
  JUPITER_ERR_CUDA = 6,         /* a CUDA runtime/driver call failed (see jupiter_last_cuda_error) */
  JUPITER_ERR_TIMEOUT = 7       /* a bounded device-side wait expired (reported by jupiter_poll_device_status) */
} jupiter_status;

/* A borrowed KV cache (Sec. II-A "KVCache").  k and v have the same geometry. */
typedef struct {
  void* k;              /* device, bf16 */
  void* v;              /* device, bf16 */
  int32_t batch;        /* sequences (prefill) or branches (suffix cache); 1 for a shared prefix */
  int32_t kv_heads;
  int32_t capacity;     /* rows per (batch, head) */
  int32_t head_dim;     /* 64 or 128 */
  int64_t stride_batch; /* elements */
  int64_t stride_head;  /* elements */
  int64_t stride_row;   /* elements, >= head_dim */
} jupiter_kv_cache;

/* Create a context on CUDA device `device`.  Allocates `workspace_bytes` of
 * device scratch (0 = a default of 64 MiB) used for split-KV partial results
 * (its first 64 KiB are completion counters, zeroed here), plus a device status
 * word.  This is the only call that allocates. */
jupiter_status jupiter_create(jupiter_ctx** out_ctx, int device, size_t workspace_bytes);

/* Frees the ctx and its scratch.  The caller must have synchronised the stream. */
void jupiter_destroy(jupiter_ctx* ctx);

const char* jupiter_status_string(jupiter_status s);

/* Text of the last CUDA error seen by this ctx ("" if none).  Host pointer, owned by the ctx. */
const char* jupiter_last_cuda_error(const jupiter_ctx* ctx);

/* Synchronises `stream`, then returns JUPITER_ERR_TIMEOUT if any kernel of this
 * ctx gave up on a bounded wait since the last poll (and clears the word),
 * JUPITER_ERR_CUDA if the stream reports an error, else JUPITER_OK. */
jupiter_status jupiter_poll_device_status(jupiter_ctx* ctx, void* stream);

/* Failure-detection aid; the paper has no counterpart.  Every device-side wait of the tensor-core kernels
 * (on a TMA copy, on a tensor-core result) is bounded: when its limit of SM clocks runs out the kernel sets the
 * ctx status word, waits for its own copies in flight, frees its tensor memory and returns normally.  From then on
 * and until jupiter_poll_device_status has reported JUPITER_ERR_TIMEOUT (which clears the word), kernels of this
 * ctx that have to wait give up as well, and the outputs of those launches are undefined.
 * This call enqueues one tiny kernel whose single wait is on a barrier that nobody arrives at, with a limit of
 * `limit_cycles` SM clocks (1 .. 2e9; JUPITER_ERR_INVALID_ARG otherwise): the wait runs out, the status word
 * is set and the kernel returns -- nothing faults, the context and the GPU stay usable.  It lets a caller (and
 * the tests) exercise the reporting path: the next jupiter_poll_device_status returns JUPITER_ERR_TIMEOUT once,
 * later polls JUPITER_OK, and later calls compute as usual. */
jupiter_status jupiter_wait_probe(jupiter_ctx* ctx, int64_t limit_cycles, void* stream);

/* Number of this library's kernel launches enqueued through the ctx so far. */
uint64_t jupiter_launch_count(const jupiter_ctx* ctx);

/* Measurement aid; the paper has no counterpart.  Enqueues a kernel that only reads the
 * `bytes` bytes at `src` (device memory, 16-byte aligned, `bytes` a multiple of 16; else
 * JUPITER_ERR_ALIGNMENT) with 16-byte loads from two full CTAs per SM.  `out` is one
 * device word owned by the caller; it is incremented only if the XOR of all words read equals
 * a fixed constant, so in practice it is left alone.  The branch-attention kernels are bound
 * by how fast a step's K/V bytes reach the SMs; timing this call on the same number of bytes
 * in the same launch chain gives that bound.  Nothing is retained after the call. */
jupiter_status jupiter_read_probe(jupiter_ctx* ctx, const void* src, size_t bytes, uint32_t* out, void* stream);

/* KVCache write (Sec. II-A; Sec. V-A step 3: candidates' K/V are stored in the
 * cache).  Copies rows t = 0..n_rows-1 of k_new / v_new ([batch][n_rows][kv_heads][D],
 * bf16, dense) into cache rows pos_b + t of every (sequence b, head), bit-exactly.
 * pos_b = d_pos[b] if d_pos (device int32[batch]) is non-NULL, else `pos`.
 * Host checks pos + n_rows <= capacity (and, with d_pos, n_rows <= capacity);
 * a device position that would run past the capacity skips that sequence's copy.
 * Nothing else in the cache is written. */
jupiter_status jupiter_kv_append(jupiter_ctx* ctx, const jupiter_kv_cache* cache, const void* k_new,
                                 const void* v_new, int32_t n_rows, int32_t pos, const int32_t* d_pos,
                                 void* stream);

/* KVCache compaction after token-tree verification (Sec. V-A, Fig. 7 step 5: the stages
 * remove the rejected candidate tokens from the KVCache).  With a chain of drafts the accepted
 * tokens are the first rows of the block and the caller simply passes a smaller length to the
 * next call; with a token tree the accepted root-to-leaf path is scattered over the block.
 * For every sequence b of `cache` (all kv heads, K and V, bit-exactly):
 *     row d_pos[b] + j  <-  row d_pos[b] + d_accept[b * q_len + j]      for j < d_n_accept[b],
 * as if all sources were read before any row is written.  No other row is written.
 *   d_pos (device int32[batch]): first row of the draft block;  q_len: its rows, 1..16
 *   (JUPITER_ERR_UNSUPPORTED above 16);  d_accept (device int32[batch][q_len]): the accepted
 *   nodes in block order, strictly increasing;  d_n_accept (device int32[batch]): their count.
 * Device values are never trusted with an address: a count outside [0, q_len] is clamped, an
 * index outside [0, q_len) moves nothing, a block that would leave the capacity skips its
 * sequence.  The new length of sequence b is d_pos[b] + d_n_accept[b] (kept by the caller). */
jupiter_status jupiter_kv_compact(jupiter_ctx* ctx, const jupiter_kv_cache* cache, int32_t q_len,
                                  const int32_t* d_pos, const int32_t* d_accept, const int32_t* d_n_accept,
                                  void* stream);

/* Chunked-prefill attention (Sec. IV-A, Fig. 5(b)).  q: [batch][q_len][q_heads][D]
 * bf16, the chunk at positions pos..pos+q_len-1 of every sequence in `cache`.
 * Row i of head h attends to cache rows 0..pos+i (inclusive) of KV head h/G with
 * softmax(scale * q.k).  Precondition: cache rows [0, pos+q_len) are valid (the
 * chunk was appended first); rows above are never read into a result.
 * out: [batch][q_len][q_heads][D] fp32.  lse (nullable): [batch][q_heads][q_len]
 * fp32, natural-log sum of exp of the scaled scores. */
jupiter_status jupiter_chunk_prefill_attn(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* cache,
                                          int32_t q_heads, int32_t q_len, int32_t pos, float scale,
                                          float* out, float* lse, void* stream);

/* KVCache write and chunked-prefill attention of one chunk in one call (Sec. II-A: a sub-sequence's
 * keys and values are stored in the KVCache as it is processed; Sec. IV-A, Fig. 5(b): it attends
 * the cached sub-sequences before it).  Same result, in `out`, `lse` and the cache, as
 *   jupiter_kv_append(ctx, cache, k_new, v_new, q_len, pos, NULL, stream) followed by
 *   jupiter_chunk_prefill_attn(ctx, q, cache, q_heads, q_len, pos, scale, out, lse, stream):
 * k_new / v_new ([batch][q_len][kv_heads][D] bf16, dense, device) are copied bit-exactly into cache
 * rows [pos, pos+q_len) of every (sequence, head) and nothing else in the cache is written; row i
 * of head h attends cache rows 0..pos-1 and the chunk's own rows 0..i.  With head_dim 128 and
 * scale > 0 this is one kernel launch (the attention reads the chunk's K/V from k_new / v_new, so
 * no thread waits for the copy); otherwise it enqueues the two kernels of the separate calls.
 * Precondition: cache rows [0, pos) are valid.  Arguments and errors as for the two calls. */
jupiter_status jupiter_chunk_prefill_append_attn(jupiter_ctx* ctx, const void* q, const void* k_new,
                                                 const void* v_new, const jupiter_kv_cache* cache,
                                                 int32_t q_heads, int32_t q_len, int32_t pos, float scale,
                                                 float* out, float* lse, void* stream);

/* Branch attention for outline-based parallel decoding with speculative
 * verification (Sec. V-B: branches share the prompt KVCache; Sec. V-A step 3:
 * q_len draft tokens verified in one pass).
 *   prefix: batch == 1; rows [0, prefix_len) valid; prefix_len may be 0.
 *   suffix: batch == n_branches; d_suffix_len (device int32[n_branches]) is the
 *           number of valid suffix rows of each branch INCLUDING the q_len rows
 *           of this block, so q_len <= d_suffix_len[b] <= max_suffix_len.
 *   max_suffix_len: host upper bound of d_suffix_len[] (<= suffix capacity);
 *           sizes the launch.  Device lengths outside [q_len, max_suffix_len]
 *           are clamped into it before any address is formed.
 *   q:   [n_branches][q_len][q_heads][D] bf16;  1 <= q_len <= 16.
 * Draft row i of branch b attends prefix rows [0, prefix_len) and suffix_b rows
 * 0..d_suffix_len[b]-q_len+i (causal inside the draft block).
 *   out: [n_branches][q_len][q_heads][D] fp32;  lse (nullable): [n_branches][q_heads][q_len].
 * Uses the ctx scratch for split-KV partials (JUPITER_ERR_WORKSPACE if too small). */
jupiter_status jupiter_branch_attn(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* prefix,
                                   int32_t prefix_len, const jupiter_kv_cache* suffix,
                                   const int32_t* d_suffix_len, int32_t max_suffix_len, int32_t n_branches,
                                   int32_t q_heads, int32_t q_len, float scale, float* out, float* lse,
                                   void* stream);

/* KVCache write and branch attention of one decoding / verification step in one launch (Sec. V-A
 * step 3: the candidates' K/V are stored in the KVCache and verified in the same pass).  Same
 * result, in `out`, `lse` and the suffix cache, as
 *   jupiter_kv_append(ctx, suffix, k_new, v_new, q_len, 0, d_pos, stream) with
 *   d_pos[b] = d_suffix_len[b] - q_len, followed by jupiter_branch_attn(...) with the same arguments:
 * k_new / v_new ([n_branches][q_len][kv_heads][D] bf16, dense, device) become suffix rows
 * [d_suffix_len[b] - q_len, d_suffix_len[b]) of branch b, bit-exactly, and nothing else in the cache
 * is written.  The attention reads those rows from k_new / v_new, so no thread waits for the copy.
 * A device length outside [q_len, max_suffix_len] is clamped as in jupiter_branch_attn (the rows then
 * go where the clamped length says, inside the capacity).  Other arguments and errors as there. */
jupiter_status jupiter_branch_append_attn(jupiter_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                          const jupiter_kv_cache* prefix, int32_t prefix_len,
                                          const jupiter_kv_cache* suffix, const int32_t* d_suffix_len,
                                          int32_t max_suffix_len, int32_t n_branches, int32_t q_heads,
                                          int32_t q_len, float scale, float* out, float* lse, void* stream);

/* One decoding / verification step for several decoder layers in one call (Sec. V-A, Fig. 7 steps 3-5 run in
 * every decoder layer of a stage; Sec. V-B: every layer keeps its own shared prompt KVCache and per-request
 * KVCaches).  Layer l has its own query block, K/V block, prefix cache, suffix cache and outputs; all layers have
 * the same geometry (head counts, head_dim, capacities, strides), the same branch lengths and the same scale.
 * Same result, layer by layer, as n_layers calls of jupiter_branch_append_attn -- the layers must not depend on one
 * another's outputs inside the call (their Q/K/V blocks are ready beforehand) -- but the layers share launches: with
 * few stacked query rows per kv head (decode) up to 16 layers run as ONE kernel launch, so the time between
 * dependent launches is paid once per 16 layers instead of once per layer; shapes that take the other kernels are
 * enqueued layer by layer.
 *   layers: HOST array of n_layers entries (read during the call only); prefix may be NULL when prefix_len == 0;
 *           lse may be NULL.  Other arguments and errors as for jupiter_branch_append_attn; every layer's
 *           descriptors are checked before anything is enqueued, and a layer whose geometry differs from
 *           layer 0's is JUPITER_ERR_INVALID_ARG. */
typedef struct {
  const void* q;                  /* [n_branches][q_len][q_heads][D] bf16 */
  const void* k_new;              /* [n_branches][q_len][kv_heads][D] bf16 */
  const void* v_new;
  const jupiter_kv_cache* prefix; /* batch == 1 */
  const jupiter_kv_cache* suffix; /* batch == n_branches */
  float* out;                     /* [n_branches][q_len][q_heads][D] fp32 */
  float* lse;                     /* nullable: [n_branches][q_heads][q_len] */
} jupiter_branch_layer;
jupiter_status jupiter_branch_append_attn_layers(jupiter_ctx* ctx, const jupiter_branch_layer* layers,
                                                 int32_t n_layers, int32_t prefix_len, const int32_t* d_suffix_len,
                                                 int32_t max_suffix_len, int32_t n_branches, int32_t q_heads,
                                                 int32_t q_len, float scale, void* stream);

/* Tuning and testing aid; the paper has no counterpart.  The branch calls (jupiter_branch_attn, _tree,
 * jupiter_branch_append_attn) pick one of three kernels from the shape: a streaming kernel for few stacked
 * query rows per kv head (decode), a tensor-core kernel (tcgen05 / TMEM) for many rows with head_dim 128, and a
 * general split-KV kernel.  This call pins the choice for later calls on `ctx`; JUPITER_BRANCH_AUTO restores the
 * default.  A call whose shape the pinned kernel cannot take returns JUPITER_ERR_UNSUPPORTED (the tensor-core
 * kernel needs head_dim 128, scale > 0, and either q_len * group <= 128 or a group size q_heads / kv_heads that
 * divides 128).  All three give the same result up to rounding. */
typedef enum {
  JUPITER_BRANCH_AUTO = 0,
  JUPITER_BRANCH_STREAM = 1,
  JUPITER_BRANCH_SPLIT_KV = 2,
  JUPITER_BRANCH_TENSOR_CORE = 3
} jupiter_branch_kernel;
jupiter_status jupiter_select_branch_kernel(jupiter_ctx* ctx, jupiter_branch_kernel which);

/* Prefill of a branch's own prompt against the shared prefix (Sec. V-B: every point-extending
 * request first ingests its own instruction while sharing the prompt KVCache).  Chunked-prefill
 * attention with one more KV segment in front:
 *   prefix: batch == 1, rows [0, prefix_len) valid (prefix_len may be 0: then this is
 *           jupiter_chunk_prefill_attn);
 *   cache:  the branches' own caches, batch == number of branches; the chunk occupies rows
 *           pos..pos+q_len-1 of every branch (same pos for all: branches at different positions
 *           take separate calls) and has been appended already;
 *   q: [batch][q_len][q_heads][D] bf16; out: same shape fp32; lse (nullable): [batch][q_heads][q_len].
 * Row i of branch b attends prefix rows [0, prefix_len) and cache_b rows 0..pos+i.
 * head_dim 128 and scale > 0 only (JUPITER_ERR_UNSUPPORTED otherwise); any q_len >= 1. */
jupiter_status jupiter_branch_prefill_attn(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* prefix,
                                           int32_t prefix_len, const jupiter_kv_cache* cache, int32_t q_heads,
                                           int32_t q_len, int32_t pos, float scale, float* out, float* lse,
                                           void* stream);

/* Branch attention with token-tree verification (Sec. V-A: the speculative module is the token-tree
 * algorithm; jupiter_branch_attn is its chain special case).  Same arguments, layouts and errors as
 * jupiter_branch_attn, plus
 *   d_tree_mask: device uint32[n_branches][q_len]; bit j of entry (b, i) set <=> draft row i of
 *           branch b attends draft row j of the same block (its ancestors and itself; bit i must be
 *           set, bits >= q_len are ignored).  The block's K/V rows are the last q_len valid suffix
 *           rows of the branch, in draft-row order.
 * Draft row i of branch b attends prefix rows [0, prefix_len), the suffix rows written before the
 * block, [0, d_suffix_len[b] - q_len), and the block rows selected by its mask.  A chain is the mask
 * (1 << (i + 1)) - 1.  NULL d_tree_mask is JUPITER_ERR_INVALID_ARG. */
jupiter_status jupiter_branch_attn_tree(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* prefix,
                                        int32_t prefix_len, const jupiter_kv_cache* suffix,
                                        const int32_t* d_suffix_len, const uint32_t* d_tree_mask,
                                        int32_t max_suffix_len, int32_t n_branches, int32_t q_heads,
                                        int32_t q_len, float scale, float* out, float* lse, void* stream);

/* Sequence-partition planner (Sec. IV-B "Selecting Optimal Sequence Partition", Eq. 2-4).  HOST
 * pointers throughout; no device is touched.
 *   q_table: [nx][ny] row-major, q_table[i*ny + j] = q(xs[i], ys[j]) = measured latency (any unit) of
 *            a sub-sequence of xs[i] tokens whose previous sub-sequences total ys[j] tokens; xs and
 *            ys strictly increasing.  Between grid points q is bilinearly interpolated, outside
 *            the grid it is clamped to the edge (the paper interpolates its profile; it does not
 *            say how).
 *   seq_len: prompt length; min_len: the paper's b (shorter sub-sequences are forbidden, Eq. 3);
 *   max_parts: largest number of sub-sequences tried (the paper uses 4 |D|); n_stages: |D| of Eq. 4;
 *   granularity: sub-sequence boundaries are multiples of it (1 = the paper's token-by-token
 *            iteration; seq_len must be a multiple).
 * For k = 1..max_parts the slowest-sub-sequence latency W(1->seq_len, k) is minimised by the
 * dynamic programme of Eq. 2 (ties: the first minimum, i.e. the shortest prefix), then the k with
 * the smallest Eq. 4 estimate  sum_i h_i + (n_stages - 1) * W  on its recorded split is returned.
 *   out_k: chosen number of sub-sequences; out_lengths: host int32[max_parts], first out_k entries
 *   are the sub-sequence lengths in order; out_slowest: W of the chosen split; out_latency: Eq. 4.
 * JUPITER_ERR_OUT_OF_RANGE if no split respects min_len; JUPITER_ERR_INVALID_ARG for bad sizes or
 * grids; JUPITER_ERR_UNSUPPORTED if (seq_len/granularity)^2 * max_parts exceeds 2^34 steps. */
jupiter_status jupiter_plan_sequence_partition(const float* q_table, const int32_t* xs, int32_t nx,
                                               const int32_t* ys, int32_t ny, int32_t seq_len, int32_t min_len,
                                               int32_t max_parts, int32_t n_stages, int32_t granularity,
                                               int32_t* out_k, int32_t* out_lengths, float* out_slowest,
                                               float* out_latency);

/* Size of the fixed scratch array behind jupiter_branch_attn_noalloc (16 MiB). */
#define JUPITER_NOALLOC_SCRATCH_BYTES (16u << 20)

/* Branch attention without any allocation and without a jupiter_ctx.  (The paper has no
 * counterpart to this call; it exists for the way the library is embedded.)
 *
 * Who needs it: a caller that may not allocate device memory where it computes attention --
 * for example a runtime whose memory pool has claimed the whole GPU, a plugin called on
 * threads where its host forbids allocator calls, or a server that guarantees a fixed
 * footprint once it is up.  jupiter_create() allocates the split-KV scratch with cudaMalloc;
 * this entry point instead uses a fixed array of JUPITER_NOALLOC_SCRATCH_BYTES that is part of
 * the library image (so every GPU that loads the library carries it until the process ends).
 * It calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * Same arguments, layouts, results and argument errors as jupiter_branch_attn, minus the ctx;
 * it runs on the CURRENT CUDA device (cudaSetDevice is the caller's job).  Differences:
 *   - sizes whose split-KV partials would not fit the fixed array are refused with
 *     JUPITER_ERR_WORKSPACE and nothing is enqueued.  The need is
 *     64 KiB + n_branches*q_len*q_heads * slots * (head_dim+2) * 4 bytes, slots being the number
 *     of prefix plus suffix splits (at most ceil(prefix_len/128) + ceil(max_suffix_len/128));
 *     n_branches*kv_heads may not exceed 16384.
 *   - the first call on each device looks up the device address of the array (once, under a
 *     lock) before launching; make that first call outside any stream capture.
 *   - all calls on a device share the one array, which keeps whatever the previous call left
 *     in it.  Its first 64 KiB are completion counters that start at zero and that every call
 *     returns to zero itself; the rest is overwritten before it is read, so no clearing is
 *     needed between calls.  But two calls whose kernels overlap on the GPU -- different
 *     streams, or different host threads without ordering -- race on it: serialise them.
 *   - there is no device status word to poll and no launch counter. */
jupiter_status jupiter_branch_attn_noalloc(const void* q, const jupiter_kv_cache* prefix, int32_t prefix_len,
                                           const jupiter_kv_cache* suffix, const int32_t* d_suffix_len,
                                           int32_t max_suffix_len, int32_t n_branches, int32_t q_heads,
                                           int32_t q_len, float scale, float* out, float* lse, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* JUPITER_H_ */
