/*
 * pod.h -- C ABI of the PoD decode-attention library (CUDA, sm_100a, one GPU).
 *
 * PoD ("Proximal tokens over Distant tokens") keeps the full per-layer K and V of the
 * proximal tokens of a sequence -- the first n_s ("sink") and the last n_r ("recent")
 * tokens -- and stores the keys of all other ("distant") tokens once per block of
 * consecutive layers; values are kept per layer (paper: abstract; Section 2.2).  At a decode
 * step, layer l scores proximal tokens with its own query and keys, takes the distant scores
 * from the lowest layer l_a of its block (query and keys of l_a), and applies one softmax
 * over both groups to its own values (Section 2.2, Eq. 1 and Eq. 2; Appendix C shows the
 * gate of Eq. 2 is exactly that single softmax).
 *
 * Conventions
 *   - All tensors are bf16, row-major, contiguous; pointers named "device" are CUDA device
 *     pointers owned by the caller, 16-byte aligned, valid until the stream work finishes.
 *   - Layers, sequences, heads and positions are 0-based.  Blocks are runs of group_size
 *     consecutive layers: block(l) = l / group_size, lowest layer l - l % group_size; the
 *     last block is short when group_size does not divide n_layers.
 *   - A sequence holding n tokens at a layer has sink positions [0, min(n, n_s)), recent
 *     positions [max(n_s, n - n_r), n) and distant positions [n_s, n - n_r).  The token being
 *     decoded is the last one: append its K/V with pod_cache_write, then call
 *     pod_decode_attn (Eq. 1 ranges end at n, the current token included).
 *   - q and K arrive with rotary position encoding already applied; distant scores pair
 *     the lowest layer's query with the lowest layer's keys, so no re-rotation is needed.
 *   - Calls return an int status: POD_OK (0), POD_DRY_RUN (1, host-only cache), or a
 *     negative POD_ERR_* code.  Nothing throws, nothing aborts.  After an error the cache is
 *     unchanged unless stated otherwise.
 *   - Work is enqueued on the CUDA stream passed by the caller (NULL = default stream) and
 *     is asynchronous unless stated.  All calls on one cache must be issued on one stream
 *     (or be ordered by the caller); the library keeps sequence lengths both on the host
 *     (validation, launch sizing) and on the device (read by the kernels in stream order).
 *   - A cache object is not thread-safe.
 */
#ifndef POD_H_
#define POD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define POD_OK            0
#define POD_DRY_RUN       1   /* host-only cache: arguments were valid, bookkeeping advanced, nothing launched */
#define POD_ERR_INVALID  (-1) /* null/misaligned pointer, index out of range, unsupported shape */
#define POD_ERR_CAPACITY (-2) /* write would exceed a sequence's capacity; nothing written */
#define POD_ERR_ORDER    (-3) /* block lengths differ, or lowest layer not decoded at these lengths */
#define POD_ERR_ARENA    (-4) /* caller's arena is too small or misaligned */
#define POD_ERR_CUDA     (-5) /* a CUDA runtime call failed; see pod_cache_last_cuda_error */
#define POD_ERR_DEVICE   (-6) /* a kernel's bounded wait gave up; results of that call are invalid */

/* pod_cache_bytes selector */
#define POD_BYTES_LIVE        0 /* bytes of valid rows in the PoD layout */
#define POD_BYTES_DENSE_EQUIV 1 /* bytes a per-layer K+V cache of the same lengths would hold */
#define POD_BYTES_ALLOCATED   2 /* bytes of the arena (regions at capacity + library scratch) */

/* pod_cache_read_region selector (logical regions of one sequence) */
#define POD_REGION_SINK_K 0 /* [layer][kv_head][n_s][d]            position j            */
#define POD_REGION_SINK_V 1
#define POD_REGION_RING_K 2 /* [layer][kv_head][n_r][d]            slot (p - n_s) % n_r  */
#define POD_REGION_RING_V 3
#define POD_REGION_DIST_K 4 /* [block of that head][kv_head][capacity-n_s-n_r][d] index p - n_s, key of the block's lowest layer */
#define POD_REGION_DIST_V 5 /* [layer][kv_head][capacity-n_s-n_r][d] index p - n_s       */

typedef struct pod_cache pod_cache; /* opaque: host bookkeeping + device arena */

typedef struct {
  int32_t n_layers;    /* L >= 1 */
  int32_t n_q_heads;   /* H_q: a multiple of H_kv with H_q / H_kv <= 8 (grouped-query attention) */
  int32_t n_kv_heads;  /* H_kv */
  int32_t head_dim;    /* d: 64 or 128 */
  int32_t group_size;  /* G >= 1 layers per block (G = 1: ordinary dense attention) */
  int32_t n_sink;      /* n_s >= 0 */
  int32_t n_recent;    /* n_r >= 1 */
  int32_t batch;       /* number of sequences B >= 1 */
  float   sm_scale;    /* logit scale; 0 means 1/sqrt(d) as in Eq. 1 */
  int32_t device;      /* CUDA device ordinal; -1 = host-only cache (no CUDA call is made) */
} pod_config;

/* Bytes of device memory a cache with these per-sequence capacities (tokens, [batch]) needs:
 * the regions of every sequence at capacity plus library scratch (device lengths, the
 * per-block query stash, split-K partials and, when group_size > 1, the distant logits a block's
 * lowest layer leaves for the block's other layers: 4 bytes per query head and distant token).
 * Returns 0 on invalid arguments.  Host only. */
size_t pod_cache_required_bytes(const pod_config* cfg, const int32_t* seq_capacity);

/* Creates a cache.  arena: device memory of at least pod_cache_required_bytes, 256-byte
 * aligned (one row of head_dim 128), owned by the caller and kept alive until
 * pod_cache_destroy; or NULL to let the library allocate (and later free) it with cudaMalloc.
 * The call sets the WHOLE arena to zero, the caller's included (one synchronous cudaMemset of
 * pod_cache_required_bytes: about 15 ms per 100 GB on a B200): the decode kernel's tiles may
 * reach a few rows past the rows a head holds, those logits are masked, but the rows must
 * hold finite numbers.  Rows that hold no token therefore read as zeros; lengths start at 0.
 * Synchronous.  The physical layout inside the arena is private; its logical content is what
 * pod_cache_read_region returns.  Every region starts on a multiple of 128 bytes.
 * More than 256 KV heads are accepted; KV heads 256 and above never reuse stored distant
 * logits (they score the block's keys themselves: same result, more bytes).
 * Errors: INVALID, ARENA, CUDA. */
int pod_cache_create(const pod_config* cfg, const int32_t* seq_capacity,
                     void* arena_device, size_t arena_bytes, pod_cache** out);

/* Head-wise blocks (Section 2.1, "Layer Grouping Strategy" and Algorithm 1: every head gets its own
 * partition of the layers into blocks of consecutive similar layers).  lowest_layer is a host
 * array [n_layers][n_kv_heads]: lowest_layer[l][h] = lowest layer of the block that holds layer l
 * for KV head h (all query heads of a KV head follow it).  It must describe runs of consecutive
 * layers: lowest_layer[0][h] = 0 and lowest_layer[l][h] is l or lowest_layer[l-1][h].
 * cfg->group_size is ignored by these two calls; everything else is as in pod_cache_required_bytes
 * and pod_cache_create, which are the special case lowest_layer[l][h] = l - l % group_size.
 * With head-wise blocks a layer may be the lowest of the block for some heads and not for others:
 * pod_decode_attn then needs, for every head whose block started lower, that lower layer decoded
 * at the same lengths before (POD_ERR_ORDER otherwise), exactly as for uniform blocks.
 * For POD_REGION_DIST_K the index passed to pod_cache_read_region counts the blocks of that head. */
size_t pod_cache_required_bytes_blocks(const pod_config* cfg, const int32_t* seq_capacity,
                                       const int32_t* lowest_layer);
int pod_cache_create_blocks(const pod_config* cfg, const int32_t* seq_capacity,
                            const int32_t* lowest_layer, void* arena_device, size_t arena_bytes,
                            pod_cache** out);

/* Greedy layer grouping (Algorithm 1), on the host: sim is [n_heads][n_layers][n_layers] with
 * sim[h][a][b] the similarity of the attention of layers a and b for head h (Section 2.1: 1 =
 * identical).  For each head, layer 0 opens a block; every next layer joins the current block if
 * its similarity to EVERY layer already in that block is >= threshold (the paper uses 0.5), else
 * it opens a new block.  Writes lowest_layer [n_layers][n_heads], ready for
 * pod_cache_create_blocks.  Computing sim (Section 2.1, from attention maps of a trained model) is
 * outside this library.  Errors: INVALID. */
int pod_greedy_layer_blocks(const float* sim, int n_heads, int n_layers, float threshold,
                            int32_t* lowest_layer);

/* Split of a cache over several GPUs by KV head (tensor parallelism; the paper's inference path is
 * one GPU, its only parallelism is in training: Section 3, "Implementation Details").  Every region
 * of the PoD layout, the query stash, the stored logits and the outputs are per KV head, and a head's
 * attention needs nothing from another head (Eq. 1, Eq. 2), so rank r of `world` simply owns KV heads
 * [r * H_kv / world, (r + 1) * H_kv / world) and the H_q / H_kv query heads of each: its cache is an
 * ordinary cache with those heads, built from *local; k, v, q, out of its calls are the rank's own
 * slices, contiguous [.][H_kv / world][d] and [B][H_q / world][d] (what column-parallel q/k/v
 * projections produce); the ranks' outputs are disjoint slices of [B][H_q][d] starting at query head
 * *first_q_head -- gather them, or feed them to a row-parallel output projection as they are.  No call
 * of this library communicates between GPUs, and no kernel is ever given another GPU's memory.
 * pod_shard_block_map cuts a head-wise map [n_layers][H_kv] down to the rank's columns
 * [n_layers][H_kv / world].  Byte counts of the ranks add up to those of the unsplit cache.
 * Host only.  Errors: INVALID (world does not divide H_kv, rank out of range, bad config). */
int pod_shard_config(const pod_config* full, int rank, int world, pod_config* local,
                     int32_t* first_kv_head, int32_t* first_q_head);
int pod_shard_block_map(const pod_config* full, const int32_t* lowest_layer, int rank, int world,
                        int32_t* local_lowest_layer);

/* Frees host state (and the arena if the library allocated it).  Synchronises the device. */
int pod_cache_destroy(pod_cache* c);

/* Appends n_tokens tokens to one layer of the cache (prefill, chunked prefill or decode
 * append), scattering them into the PoD layout and moving rows that leave the recent window
 * to the distant stores: values always, keys only when `layer` is the lowest layer of its
 * block, so distant keys are written once per block (reading of the paper's cache-update
 * figure, Fig. 2 right: a token is demoted when it falls out of the last n_r tokens).
 *   seq >= 0 : k, v are device bf16 [n_tokens][H_kv][d] for that sequence.
 *   seq == -1: n_tokens must be 1; k, v are device bf16 [B][H_kv][d], one token for every
 *              sequence.
 * Errors: INVALID, CAPACITY (length + n_tokens > capacity of a sequence; nothing written),
 * CUDA. */
int pod_cache_write(pod_cache* c, int layer, int seq, const void* k_device,
                    const void* v_device, int n_tokens, void* cuda_stream);

/* Decode-step attention of one layer for every sequence (Eq. 1 + Eq. 2 / Appendix C):
 *   logits of proximal tokens  = sm_scale * <q[b][h], K_layer[p][h / r]>
 *   logits of distant tokens   = sm_scale * <q_low[b][h], K_low[p][h / r]>, q_low being the q
 *                                passed to this function for the block's lowest layer at the
 *                                same step (the library stashes it), K_low the block's key store
 *   out[b][h] = softmax over all logits applied to V_layer, fp32 accumulation, bf16 result.
 * q_device, out_device: device bf16 [B][H_q][d].  A sequence of length 0 gives zeros.
 * Call order inside a decode step: layers in increasing order within a block, lowest first;
 * all layers of a block must hold the same lengths.  Errors: INVALID, ORDER, CUDA. */
int pod_decode_attn(pod_cache* c, int layer, const void* q_device, void* out_device,
                    void* cuda_stream);

/* pod_cache_write(layer, seq = -1, k, v, 1) followed by pod_decode_attn(layer, q, out), as one
 * kernel launch: the decode step of Section 2.2 as a layer runs it -- append the current token's
 * K/V, then attend over all tokens up to and including it (Eq. 1 ranges end at n) -- with the
 * cache update of Fig. 2 (right) applied by the same kernel: the new rows go to the sink or to
 * their ring slot, the slot's previous occupant moves to the distant stores (value always, key
 * from the block's lowest layer only).  Results (output and cache contents) are those of the
 * two separate calls; only the summation order of the softmax differs.
 *   k_device, v_device: device bf16 [B][H_kv][d], one new token per sequence.
 *   q_device, out_device: device bf16 [B][H_q][d].
 * Errors: INVALID, CAPACITY (a sequence is full; nothing changed), ORDER (as pod_decode_attn,
 * judged at the lengths after the append), CUDA. */
int pod_append_decode_attn(pod_cache* c, int layer, const void* k_device, const void* v_device,
                           const void* q_device, void* out_device, void* cuda_stream);

/* Gate threshold of the paper's appendix "Computation Optimization for Distant Tokens".  For a head
 * of a layer that is not the lowest layer of the head's block, the gate of Eq. 2,
 * g = sum exp(a^P) / (sum exp(a^P) + sum exp(a^D)), can be evaluated before any distant value is
 * read: a^D are the lowest layer's logits, whose sum that layer has left behind.  With a threshold
 * 0 <= tau <= 1 set, such a head omits its distant tokens when g >= tau: its output is then the
 * softmax over its proximal tokens alone (reading of "omitted": the gate is taken as 1).  Heads of
 * lowest layers, and heads that cannot use their block's stored logits (see pod_decode_attn's call
 * order), always attend to everything.  tau > 1 (the default) switches the gate off.  A gated
 * pod_decode_attn / pod_append_decode_attn of such a layer runs as two launches: the proximal
 * tokens, then the distant tokens of the KV heads in which some query head did not skip (the
 * distant values are shared by the query heads of a KV head).  The decision is taken in fp32 on
 * the device; results depend on tau by design (an approximation, as in the paper).
 * Errors: INVALID (tau negative or not a number). */
int pod_cache_set_gate_threshold(pod_cache* c, float tau);

/* Byte accounting (host integers).  Live bytes of a sequence of length n (at the layer with
 * the most tokens): row * H_kv * (L * (2 n_p + n_d) + ceil(L / G) * n_d), n_p = min(n, n_s+n_r),
 * n_d = n - n_p; the saving against dense is (n_d / n) (1 - ceil(L/G)/L) / 2 -- only keys
 * are shared (Section 2.2; Section 3 "KV Cache Memory").  Returns -1 on error. */
int64_t pod_cache_bytes(const pod_cache* c, int which);

/* Tokens currently held by (seq, layer); negative status on error.  Host only. */
int pod_cache_seq_len(const pod_cache* c, int seq, int layer);

/* Forgets the contents of one sequence (seq >= 0) or of all (seq == -1).  Synchronous. */
int pod_cache_reset(pod_cache* c, int seq);

/* Test/debug export: copies `count` rows (d bf16 each) starting at row `first` of a logical
 * region to host memory.  Synchronises the device.  Only rows that hold a token are
 * meaningful.  layer_or_block is a block index for POD_REGION_DIST_K, a layer otherwise. */
int pod_cache_read_region(const pod_cache* c, int region, int layer_or_block, int seq,
                          int kv_head, int first, int count, void* host_dst);

/* Synchronises the device and reports POD_ERR_DEVICE if any kernel of this cache hit a
 * bounded-wait limit since the last call (the flag is cleared), else POD_OK. */
int pod_cache_device_status(pod_cache* c);

/* Fault injection from the host, for tests of that error path (the paper has no counterpart): sets
 * the cache's error word as a kernel whose bounded wait gave up would, without making any kernel
 * fail.  The next pod_cache_device_status reports POD_ERR_DEVICE once and clears the word.
 * Synchronises the device.  Errors: INVALID, CUDA. */
int pod_cache_inject_error(pod_cache* c);

/* Test hook (the paper has no counterpart).  Decode launches that follow a decode launch of another layer
 * of the same cache start "optimistically": they stream with a copy of q read before the stream's
 * previous kernel is known to have finished, wait for that kernel only before they publish anything, then
 * read q again and compare; a head in which a copy turned out stale is recomputed by one CTA with a plain
 * loop (exact, slow).  That path is never taken when q is complete before the call is enqueued, so this
 * call forces it: the next pod_decode_attn / pod_append_decode_attn (not a gated one) treats every early
 * copy as stale.  Results must not change.  Errors: INVALID. */
int pod_cache_inject_stale_query(pod_cache* c);

/* Last CUDA runtime error code seen by this cache (0 if none). */
int pod_cache_last_cuda_error(const pod_cache* c);

/* Launch geometry of the most recent pod_decode_attn (diagnostics for benchmarks):
 * tokens per split, CTAs launched, and kernels launched by that call. */
int pod_cache_last_launch(const pod_cache* c, int32_t* split_tokens, int32_t* n_ctas,
                          int32_t* n_kernels);

/* Launch trace, for benchmarks (the paper has no counterpart).  Consecutive decode launches of a stream
 * overlap -- a launch requests its first tiles while the previous one finishes -- so CUDA events between
 * them (which would serialise them) cannot say what one launch of a pipelined step costs.  With a trace
 * set, each of the next n_launches kernels of pod_decode_attn / pod_append_decode_attn (a gated layer
 * is two) writes one pair of uint64 into pairs_device: the GPU's nanosecond timer when its first CTA
 * starts and when its last CTA ends.  pairs_device: device memory of n_launches * 16 bytes, 8-byte
 * aligned, caller-owned; the call initialises it (synchronously).  NULL, 0 switches the trace off.
 * pod_cache_trace_count: pairs handed out so far.  Cost when on: two atomics per CTA.
 * Errors: INVALID, CUDA. */
int pod_cache_set_trace(pod_cache* c, void* pairs_device, int n_launches);
int pod_cache_trace_count(const pod_cache* c);

const char* pod_strerror(int status);

/* PoD attention for every position of a sequence (prefill; Section 2.2, Eq. 1, Eq. 2 and the masks of
 * Fig. 2, middle), from the layer's dense projections, on the tcgen05 tensor cores.  Position i attends
 * to positions j <= i; of those the first n_sink and the last n_recent (i included) are proximal, with
 * logits sm_scale <q[i][h], k[j][h / r]>; the others are distant, with logits
 * sm_scale <q_low[i][h], k_low[j][h / r]>, q_low / k_low being the queries and keys of the lowest layer
 * of the head's block.  out[i][h] = one softmax over both groups applied to v.  It is what
 * pod_decode_attn returns at each step of a sequence fed token by token.
 *   q, q_low, out : device bf16 [n_tokens][n_q_heads][head_dim];  k, k_low, v : device bf16
 *                   [n_tokens][n_kv_heads][head_dim]; head_dim 64 or 128.
 *   q_low, k_low  : NULL for a layer that is the lowest of every head's block (ordinary causal attention).
 *   head_shares   : host int32 [n_kv_heads] or NULL; with q_low given, KV head h takes its distant logits
 *                   from q_low / k_low if head_shares is NULL or head_shares[h] != 0 (head-wise blocks).
 * The cache is not touched: write k, v with pod_cache_write.  Runs on the current device; the first call
 * on a device looks up the driver's tensor-map encoder and the address of the status word (a word inside the
 * library's device image: nothing is allocated).  With q_low given at most 256 KV heads (INVALID beyond).
 * Asynchronous on cuda_stream.  Errors: INVALID, CUDA.  pod_prefill_status synchronises the device and returns
 * POD_ERR_DEVICE if a launch gave up a bounded wait since the last call (its output is then invalid;
 * until this call has read the error, further launches on the device return without computing). */
int pod_prefill_attn(int n_tokens, int n_q_heads, int n_kv_heads, int head_dim, int n_sink, int n_recent,
                     float sm_scale, const void* q_device, const void* k_device, const void* v_device,
                     const void* q_low_device, const void* k_low_device, const int32_t* head_shares,
                     void* out_device, void* cuda_stream);
int pod_prefill_status(void);
/* Fault injection from the host, for tests of that error path (the paper has no counterpart): sets the error
 * word of the current device as a launch whose wait gave up would.  Until pod_prefill_status has read it,
 * pod_prefill_attn launches on the device return without writing their output.  Synchronises the device.
 * Errors: INVALID before the first pod_prefill_attn on the device, CUDA. */
int pod_prefill_inject_error(void);

/* Decode attention without any allocation.  (The paper has no counterpart of this call; it is a
 * packaging variant of pod_decode_attn for one sequence of ordinary, unshared K/V.)
 *
 * Some programs that embed this library cannot obtain device memory at the moment they need
 * attention: a serving process whose own memory pool has already claimed the whole GPU, so a
 * raw cudaMalloc would fail; a plug-in running under a host framework that forbids allocating
 * behind its back; a latency-critical loop that cannot afford the implicit device-wide
 * synchronisation an allocation or a free may cause.  pod_cache_create needs an arena with
 * room for the split-K partial results; this call needs none.  Its partials live in a fixed
 * array inside the library's device image (POD_STATIC_SCRATCH_BYTES, about 2.1 MB, held by
 * every GPU that loads the library until the process exits).  It calls no cudaMalloc, no
 * cudaFree and no allocating library routine.
 *
 *   kv_device : device bf16 [2][n_kv_heads][capacity][head_dim]: all keys, then all values,
 *               head-major, token p of head h at row p.  Rows at or past n_tokens (up to the
 *               next multiple of 16) are loaded and masked, so they must hold finite numbers:
 *               zero the buffer once when it is created.
 *   q_device  : device bf16 [n_q_heads][head_dim];  out_device: device bf16, same shape.
 *   out[h] = softmax_p(sm_scale <q[h], K[p][h / r]>) V[.][h / r] over p < n_tokens (zeros when
 *   n_tokens == 0); sm_scale 0 means 1/sqrt(head_dim).  Runs on the current device.
 *
 * Limits (POD_ERR_CAPACITY beyond them): n_q_heads <= 64, n_tokens <= capacity,
 * 2 * n_kv_heads * capacity < 2^31.  Shapes as for pod_config (head_dim 64 or 128, at most 8
 * query heads per KV head); other invalid arguments give POD_ERR_INVALID.
 *
 * The pointers must belong to the current device.  The first call on each device looks up the array's
 * device address (cudaGetSymbolAddress) and the driver's tensor-map encoder, sets the kernel's
 * shared-memory attribute on that device and zeroes the error word; make that first call outside any
 * stream capture.  All calls
 * on a device share the one array, which keeps the previous call's contents; the call clears
 * the counters that must start at zero on the given stream.  Two calls whose kernels may run at
 * the same time on one device (different streams, different threads) race on the array: order
 * them.  Asynchronous on cuda_stream like pod_decode_attn. */
#define POD_STATIC_SCRATCH_BYTES 2171136
int pod_dense_decode_attn_static(const void* kv_device, int capacity, int n_tokens,
                                 const void* q_device, void* out_device, int n_q_heads,
                                 int n_kv_heads, int head_dim, float sm_scale, void* cuda_stream);
/* Error word of the fixed array on the current device (the paper has no counterpart): synchronises the
 * device and returns POD_ERR_DEVICE if a pod_dense_decode_attn_static kernel gave up a bounded wait since
 * the last call (the outputs of the calls since then are invalid), else POD_OK; the word is cleared.  The
 * calls themselves never clear it.  No allocation: one small copy through the array's address.  Call it with
 * the device current that ran the kernels.  ..._inject_error sets the word from the host (tests of this
 * path; no kernel is made to fail).  Errors: CUDA. */
int pod_dense_decode_attn_static_status(void);
int pod_dense_decode_attn_static_inject_error(void);

#ifdef __cplusplus
}
#endif
#endif /* POD_H_ */
