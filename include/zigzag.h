/*
 * zigzag.h -- C ABI of the ZigzagAttention inference hot path for NVIDIA B200 (sm_100a).
 *
 * The library runs the per-layer attention pass of a model whose layers are each
 * exclusively "retrieval" (full causal attention over the whole KV cache) or
 * exclusively "streaming" (attention to sink tokens plus a recent window, the rest of
 * the KV waived), so that each layer needs one attention call (paper: Introduction,
 * last-but-one paragraph; Section 2.2, first paragraph).  It also carries the
 * DuoAttention-style layer that mixes both kinds of head in one layer and therefore
 * runs two passes plus head gather/scatter (paper: Introduction, the paragraph on the
 * cost of DuoAttention; Section 2.1, last paragraph) as the in-library comparison.
 *
 * Conventions
 *   - Every function returns an int status: ZZ_OK (0) or a negative ZZ_ERR_* code.
 *     Nothing throws or aborts across this boundary.  A call that fails argument or
 *     capacity validation has launched nothing and leaves the cache unchanged.
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller
 *     allocates and owns all device memory (tensors, the cache arena, the workspace);
 *     the library owns only the small host-side handle.  Unless stated otherwise the
 *     library never allocates or frees device memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All
 *     compute calls are asynchronous on that stream.  A handle is not thread-safe and
 *     calls on one handle must be issued in stream order on one stream at a time.
 *   - Tensors are bf16 (2-byte), row-major, innermost dimension head_dim (128, or 64; the sizes
 *     written as 128 below are head_dim).
 *     q/out of a call:   [tokens, n_q_heads, head_dim]
 *     k/v of a call:     [tokens, n_kv_heads, head_dim]
 *     `tokens` is the packed concatenation over the batch, sequence 0 first.
 *   - Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   - Token positions are absolute and 0-based; a sequence's length `len` is the number
 *     of tokens appended so far.  Lengths live on the device (so that a captured
 *     sequence of calls can be replayed) and are mirrored on the host for validation.
 *
 * Visibility rule (S = sink, W = recent):
 *   retrieval head:  the query at position t sees every key j <= t;
 *   streaming head:  it sees key j <= t iff  j < S  or  t - j < W  (the window counts
 *                    the current token).
 * Streaming KV store: a ring of S+W slots per (layer, sequence, KV head);
 *   slot(t) = t for t < S, else S + ((t - S) mod W); pos[slot] is the token held or -1.
 * Retrieval KV store: slot j holds token j, up to capacity[seq] tokens.
 */
#ifndef ZIGZAG_H_
#define ZIGZAG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ZZ_OK 0
#define ZZ_ERR_INVALID_ARG (-1) /* NULL pointer, index out of range, inconsistent sizes        */
#define ZZ_ERR_UNSUPPORTED (-2) /* head_dim not 64 or 128, group size > 16, batch > ZZ_MAX_BATCH,
                                   FP8 or paged stores at head_dim 64, ...                      */
#define ZZ_ERR_CAPACITY (-3)    /* len + n_new would exceed capacity[seq] of a retrieval store  */
#define ZZ_ERR_WORKSPACE (-4)   /* arena or workspace smaller than zz_cache_query reported      */
#define ZZ_ERR_CUDA (-5)        /* a CUDA runtime/driver call failed                            */
#define ZZ_ERR_TIMEOUT (-6)     /* a bounded device-side wait expired (see zz_get_last_status)  */

#define ZZ_MAX_BATCH 64
#define ZZ_KIND_STREAMING 0
#define ZZ_KIND_RETRIEVAL 1

typedef struct zz_cache zz_cache_t;

/* Plain-data description of the attention stack.  All pointers are HOST pointers and
 * are only read during zz_cache_query / zz_cache_create. */
typedef struct zz_config {
    int32_t n_layers;
    int32_t batch;                      /* sequences, 1 .. ZZ_MAX_BATCH                         */
    int32_t n_q_heads;
    int32_t n_kv_heads;                 /* divides n_q_heads; group size <= 16                  */
    int32_t head_dim;                   /* 128 or 64 (FP8 and paged stores: 128 only)           */
    int32_t sink;                       /* S >= 0                                               */
    int32_t recent;                     /* W >= 1                                               */
    int32_t max_new_tokens;             /* largest sum of n_new over the batch in one prefill
                                           call (sizes the mixed-layer gather buffers); >= batch */
    float softmax_scale;                /* e.g. 1/sqrt(128)                                     */
    const uint8_t* layer_is_retrieval;  /* [n_layers]  the exclusive per-layer mask             */
    const uint8_t* kvhead_is_retrieval; /* NULL, or [n_layers * n_kv_heads]: per-KV-head kinds
                                           (overrides the layer mask; a layer holding both
                                           kinds runs the two-pass mixed-head path)             */
    const int32_t* capacity;            /* [batch] max tokens per sequence in retrieval stores  */
    int32_t retrieval_kv_fp8;           /* 0: retrieval stores hold the bf16 rows as given; 1: they
                                           hold FP8 rows (see "FP8 retrieval stores" below)        */
} zz_config_t;

/* Library version (major*10000 + minor*100 + patch). */
int zz_version(void);
/* Static, NUL-terminated description of a status code. */
const char* zz_status_str(int status);

/* Bytes the caller must provide for the KV arena and the workspace (both device memory,
 * 256-byte aligned).  Cache layout: paper, Introduction (KV cache of the prefill and decoding phases); streaming
 * stores keep only sink + recent entries (Introduction; Section 3.3 for the sizes). */
int zz_cache_query(const zz_config_t* cfg, size_t* arena_bytes, size_t* workspace_bytes);

/* Builds the handle on caller-provided device memory, zero-fills the arena, sets all
 * lengths to 0 and all ring positions to -1.  Synchronous (returns after the device
 * finished initialising).  *out is written only on success. */
int zz_cache_create(const zz_config_t* cfg, void* d_arena, size_t arena_bytes, void* d_workspace,
                    size_t workspace_bytes, zz_cache_t** out);
/* Paged retrieval stores (a variant the paper does not describe; the attention computed is the
 * same).  The retrieval stores of all layers and sequences share one pool of `pool_pages` pages;
 * a page holds 128 tokens of one KV head (its K rows, then its V rows: 64 KB).  A sequence takes
 * pages as it grows (one per retrieval KV head of the layer per 128 tokens) and returns them in
 * zz_cache_reset, so the pool may be smaller than the sum of the capacities; capacity[seq] stays
 * the most tokens a sequence may hold (it sizes the page table).  Calls that add tokens
 * (zz_kv_append, zz_decode_step, zz_decode_step_all, the *_host entries, zz_cache_import) return
 * ZZ_ERR_CAPACITY, having launched and changed nothing, when the pool has too few free pages.
 * Streaming rings are not paged.  Page bookkeeping lives on the host; its device-side table is
 * written by small launches on the caller's stream, so one handle must be driven from one stream
 * at a time.  Everything else behaves as with zz_cache_query / zz_cache_create. */
int zz_cache_query_paged(const zz_config_t* cfg, int32_t pool_pages, size_t* arena_bytes, size_t* workspace_bytes);
int zz_cache_create_paged(const zz_config_t* cfg, int32_t pool_pages, void* d_arena, size_t arena_bytes,
                          void* d_workspace, size_t workspace_bytes, zz_cache_t** out);
/* Pages of the pool and pages free now (both 0 for a cache with contiguous stores). */
int zz_cache_pages(const zz_cache_t* cache, int32_t* total, int32_t* free_now);
/* Replaying decode steps from a CUDA graph.  zz_decode_step / zz_decode_step_all may be captured
 * into a graph (they only launch kernels); a replay repeats the launch plan of the capture, the
 * kernels take the lengths from device memory, and the last split of each sequence absorbs the
 * tokens added since the capture (re-capture every few hundred steps to keep the splits even).
 * The host does not see replays, so: (1) before capturing, call zz_cache_reserve with the number
 * of steps that will be replayed: it checks the capacities and, for a paged cache, takes the
 * pages now (ZZ_ERR_CAPACITY, nothing changed, if they do not fit); (2) after the replays, call
 * zz_cache_sync_len, which reads the device lengths back into the host mirror (it synchronises
 * the stream).  A replay that runs out of room anyway is refused on the device: the kernels of
 * that sequence's retrieval layers store and write nothing and zz_get_last_status returns
 * ZZ_ERR_CAPACITY (the sequence is then inconsistent across layers: reset it).  The capture call
 * itself counts as one step in the host mirror but executes nothing. */
int zz_cache_reserve(zz_cache_t* cache, int32_t extra_tokens, void* stream);
int zz_cache_sync_len(zz_cache_t* cache, void* stream);
/* Frees the host handle (device memory stays the caller's). */
int zz_cache_destroy(zz_cache_t* cache);
/* Forgets the tokens of sequence `seq` (-1: all sequences) in every layer. */
int zz_cache_reset(zz_cache_t* cache, int seq, void* stream);
/* Host-mirrored length of (layer, seq). */
int zz_cache_len(const zz_cache_t* cache, int layer, int seq, int32_t* len);

/* Tuning knobs for experiments; the paper has no counterpart.  Keys: "decode_min_chunk"
 * (fewest tokens per split of the long-store decode plan; a multiple of 16, default 256);
 * "decode_short_tokens" (tokens per CTA of the short-store plan, and the threshold
 * total_tokens * kv_heads <= SMs * value below which it is used; multiple of 16, default
 * 384; 0 disables the short-store plan); "decode_overlap" (how the layers
 * of zz_decode_step_all are launched.  3, the default: all exclusive retrieval layers in one
 * launch and all exclusive streaming layers in another; the mixed layers, if they all have the
 * same number of retrieval heads, in one launch per pass plus one head-regrouping copy before and
 * one after (possible when all layers hold equally long sequences; otherwise as 2, with the
 * four launches of a mixed layer in plain order); 2: one launch per layer, programmatic
 * dependent launch and no wait between layers -- they share no scratch, so a layer's kernel fills
 * the SMs the previous one leaves idle; 1: the same, but each kernel waits for the previous one
 * before it merges; 0: plain stream order); "decode_multi_waves" (default 8: a grid over n layers
 * cuts every layer into about 2 * SMs * value / n work items instead of 2 * SMs). */
int zz_tune(zz_cache_t* cache, const char* key, int value);

/* KV append with sink + recent eviction (paper: Introduction -- the KV cache grows with
 * the tokens seen; streaming heads waive all but sink and recent entries).
 * Appends h_n_new[b] tokens of sequence b to `layer`: retrieval stores take token t in
 * slot t; streaming stores take it in slot(t), overwriting token t - W.  d_k/d_v are
 * packed [sum n_new, n_kv_heads, 128].  Fails with ZZ_ERR_CAPACITY (nothing written)
 * if any retrieval store would overflow. */
int zz_kv_append(zz_cache_t* cache, int layer, const void* d_k, const void* d_v,
                 const int32_t* h_n_new, void* stream);

/* Prefill attention of one layer (paper: Introduction, prefilling phase; Section 2.1, the
 * two kinds of attention).  For sequence b the h_n_new[b] new queries sit at positions
 * len .. len+n_new-1 and attend over (the store as it stands) U (the new chunk d_k/d_v)
 * under the visibility rule of their head's kind.  The store is NOT modified: append the
 * same chunk afterwards with zz_kv_append (attend-then-append, so a chunk longer than the
 * window never evicts keys its own early rows need).  d_q/d_out are packed
 * [sum n_new, n_q_heads, 128]; d_k/d_v packed [sum n_new, n_kv_heads, 128]; all four must
 * be 16-byte aligned. */
int zz_prefill_attn(zz_cache_t* cache, int layer, const void* d_q, const void* d_k,
                    const void* d_v, void* d_out, const int32_t* h_n_new, void* stream);

/* Decode attention of one layer (paper: Introduction, decoding phase): one query per
 * sequence, at position len-1, over the store, which must already hold that token.
 * d_q/d_out: [batch, n_q_heads, 128]. */
int zz_decode_attn(zz_cache_t* cache, int layer, const void* d_q, void* d_out, void* stream);

/* zz_kv_append of one token per sequence followed by zz_decode_attn. */
int zz_decode_step(zz_cache_t* cache, int layer, const void* d_q, const void* d_k,
                   const void* d_v, void* d_out, void* stream);

/* One decode step of the whole stack: the result of zz_decode_step for every layer, with the
 * q/k/v of all layers given up front (d_q/d_out: [n_layers, batch, n_q_heads, 128]; d_k/d_v:
 * [n_layers, batch, n_kv_heads, 128]), which lets the layers share launches (see "decode_overlap"
 * under zz_tune).  Capacity is validated for every layer before anything is launched. */
int zz_decode_step_all(zz_cache_t* cache, const void* d_q, const void* d_k, const void* d_v,
                       void* d_out, void* stream);

/* The same two calls fed from HOST memory: copies q/k/v into caller-provided device
 * staging (d_stage, at least zz_stage_bytes(cache, n_tokens) bytes), runs the call and
 * copies the result back to h_out.  Pinned host memory makes the copies asynchronous.
 * Prefill also appends the chunk after attending. */
size_t zz_stage_bytes(const zz_cache_t* cache, int64_t n_tokens);
int zz_decode_step_host(zz_cache_t* cache, int layer, const void* h_q, const void* h_k,
                        const void* h_v, void* h_out, void* d_stage, size_t stage_bytes,
                        void* stream);
/* zz_decode_step_all fed from HOST memory: h_q/h_out [n_layers, batch, n_q_heads, 128], h_k/h_v
 * [n_layers, batch, n_kv_heads, 128]; d_stage holds at least
 * zz_stage_bytes(cache, n_layers * batch) bytes.  When h_q, h_k and h_v lie back to back in host
 * memory (in that order) they travel in one copy. */
int zz_decode_step_all_host(zz_cache_t* cache, const void* h_q, const void* h_k, const void* h_v,
                            void* h_out, void* d_stage, size_t stage_bytes, void* stream);
int zz_prefill_host(zz_cache_t* cache, int layer, const void* h_q, const void* h_k,
                    const void* h_v, void* h_out, const int32_t* h_n_new, void* d_stage,
                    size_t stage_bytes, void* stream);

/* FP8 retrieval stores (cfg.retrieval_kv_fp8 = 1; a variant the paper does not describe -- its
 * motivation, the size of the KV cache, is the Introduction's second paragraph).  Every row that
 * enters a retrieval store (one token, one KV head, K or V) is stored as 128 codes in the 8-bit
 * floating-point format E4M3 (1 sign, 4 exponent bits of bias 7, 3 mantissa bits, largest magnitude
 * 448, no infinities) plus one scale byte e that stands for 2^(e - 127):
 *   amax = the row's largest magnitude = m * 2^k, 1 <= m < 2;  e = k + 127 - 8 (+ 1 if m > 1.75),
 *   at least 1: the smallest power of two that brings amax to at most 448, so nothing saturates;
 *   code = the E4M3 number nearest to x / 2^(e-127), ties to the even code.
 * The stored value is code * 2^(e-127), exactly, and attention over the store uses those values:
 * 258 bytes per token and head instead of 512.  Queries, probabilities and accumulation are as
 * with bf16 stores.  What attends to what: a decode step stores its token first, so the query
 * sees its own token as stored; a prefill chunk sees earlier tokens as stored and its own tokens
 * as given (bf16), and is stored afterwards by zz_kv_append.  Streaming rings stay bf16.  Not
 * available together with paged stores (ZZ_ERR_UNSUPPORTED).  zz_cache_export / zz_cache_import
 * refuse the retrieval group of such a cache (ZZ_ERR_UNSUPPORTED); the two calls below move its
 * bytes: h_k_codes/h_v_codes [n_retrieval_heads, capacity[seq], 128] uint8 and h_k_scale/h_v_scale
 * [n_retrieval_heads, capacity[seq]] uint8, heads in ascending KV-head order, slot j = token j.
 * Both synchronise the stream. */
int zz_cache_export_fp8(zz_cache_t* cache, int layer, int seq, void* h_k_codes, void* h_v_codes,
                        void* h_k_scale, void* h_v_scale, int32_t* h_len, void* stream);
int zz_cache_import_fp8(zz_cache_t* cache, int layer, int seq, const void* h_k_codes, const void* h_v_codes,
                        const void* h_k_scale, const void* h_v_scale, int32_t len, void* stream);

/* Snapshot of one store, for tests and checkpointing.  `kind` selects the KV-head group
 * of the layer (ZZ_KIND_RETRIEVAL / ZZ_KIND_STREAMING; an exclusive layer has only one).
 * h_k/h_v receive [n_heads_of_kind, n_slots, 128] bf16 in ascending KV-head order, where
 * n_slots = capacity[seq] (retrieval) or S+W (streaming); h_pos [n_slots] receives the
 * token held by each slot or -1; *h_len the length.  zz_cache_export_shape reports
 * n_heads_of_kind and n_slots.  Both synchronise the stream. */
int zz_cache_export_shape(const zz_cache_t* cache, int layer, int seq, int kind,
                          int32_t* n_heads, int32_t* n_slots);
int zz_cache_export(zz_cache_t* cache, int layer, int seq, int kind, void* h_k, void* h_v,
                    int32_t* h_pos, int32_t* h_len, void* stream);
/* Inverse of zz_cache_export for one group; sets the length of (layer, seq) to `len`. */
int zz_cache_import(zz_cache_t* cache, int layer, int seq, int kind, const void* h_k,
                    const void* h_v, const int32_t* h_pos, int32_t len, void* stream);

/* Reads (and clears) the device status word: ZZ_OK, ZZ_ERR_TIMEOUT if a bounded wait inside a
 * kernel expired since the last read, ZZ_ERR_CAPACITY if a replayed decode step found a retrieval
 * store full, ZZ_ERR_UNSUPPORTED if a decode launch was refused for a split plan beyond the
 * kernel's limit.  Synchronises the stream. */
int zz_get_last_status(zz_cache_t* cache, void* stream);

/* Self-test of the failure path of the kernels' bounded waits (the paper has no counterpart).
 * Every wait inside the kernels (on a shared-memory barrier that a copy or an MMA completes) gives
 * up after a fixed number of probes, records ZZ_ERR_TIMEOUT in the status word and lets the
 * kernel return, so a wait that can never end costs a status instead of a hung device.  This
 * call launches one warp that runs that same wait on a barrier nothing ever completes, with the
 * limit set to max_polls (1 .. 65536) and no copy or MMA in flight; it returns ZZ_OK once the
 * kernel has given up and returned (it synchronises the stream), and the next
 * zz_get_last_status then reports ZZ_ERR_TIMEOUT.  The device context stays usable. */
int zz_selftest_wait_timeout(zz_cache_t* cache, int32_t max_polls, void* stream);

/* Tracer (the paper has no counterpart; it reports per-token latencies only, Section 3.2).
 * zz_profile_enable(n): n = 0 switches it off; n >= 1 brackets every n-th launch of each
 * kernel class with two CUDA events on its stream (sampling keeps the host overhead low).
 * zz_profile_read waits for the recorded events of one kernel class, returns how many
 * launches were recorded and their summed device time, and (reset != 0) forgets all records.
 * Classes: 0 append, 1 decode retrieval, 2 decode streaming, 3 prefill retrieval,
 * 4 prefill streaming, 5 head regroup.  Process-wide, not thread-safe. */
int zz_profile_enable(int period);
int zz_profile_read(int kind, int64_t* launches, double* total_ms, int reset);

/* Decode attention without any workspace from the caller (the paper has no counterpart: this
 * is a deployment convenience, not part of the method).
 *
 * For callers that cannot allocate device memory -- a server that has given the whole device
 * to its own pool, a plug-in whose host forbids allocations after start-up -- and therefore
 * cannot hand the library a workspace.  The scratch the split-sequence decode kernel needs
 * (partial outputs, their softmax statistics, arrival counters, the device copy of the lengths)
 * lives in a fixed array of about 2.1 MB inside the library's device image; every GPU that loads
 * the library holds it until the process exits.  The call itself never calls cudaMalloc, cudaFree
 * or any allocating routine.  (Loading the library's device image is the CUDA runtime's business:
 * with lazy module loading it happens at the first call on a device, and that is when the driver
 * sets the array and the kernels up.  Make that first call at start-up, before the caller's own
 * pool claims what is left of the device; every later call touches no allocator at all.)
 *
 * Computes, for each sequence b, full (retrieval) attention of one query token over the first
 * h_len[b] rows of the caller's stores:
 *   d_q, d_out  [batch, n_q_heads, 128] bf16 (device)
 *   d_k, d_v    [batch, n_kv_heads, capacity, 128] bf16 (device), row j = token j
 *   h_len       [batch] int32 (host), 1 <= h_len[b] <= capacity
 * Limits, fixed by the size of the array: batch <= 16 and batch * n_q_heads <= 64; anything
 * larger is refused with ZZ_ERR_WORKSPACE before anything is launched (the limits can be read
 * with zz_decode_attn_static_limits).  Group size and head_dim rules are the library's usual ones.
 *
 * The first call on a device looks up the array's device address (and opts the kernel into its
 * shared-memory size); make that first call outside any stream capture.  All calls, from every
 * thread and stream, share the one array per device: it keeps the previous call's contents (the
 * call clears the counters it needs at zero itself), and two calls whose kernels may overlap on
 * the GPU race on it -- issue them on one stream, or order them yourself.  Asynchronous on
 * `stream`: each call enqueues a copy of h_len and bakes the split plan it derives from h_len
 * into the launch, so h_len may be reused as soon as the call returns if it is pageable memory,
 * and after the stream reaches the copy if it is pinned. */
int zz_decode_attn_static(const void* d_q, const void* d_k, const void* d_v, void* d_out,
                          const int32_t* h_len, int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                          int32_t capacity, float softmax_scale, void* stream);
int zz_decode_attn_static_limits(int32_t* max_batch, int32_t* max_batch_times_q_heads,
                                 size_t* scratch_bytes);

/* Layer-mask solver (paper: Section 2.2 "Transport Optimization", Eq. 5; the quantile split it
 * starts from is the last paragraph of Section 2.1).  Host function, no device work.
 *   h_alpha [n_layers * n_heads]  per-head importances (the converged alpha of the head-importance
 *                                 training; larger = needs full attention), finite
 *   n_streaming_layers = p        layers that become all-streaming; the quantile split marks the
 *                                 p * n_heads heads of smallest alpha as streaming heads (sparsity p / L)
 *   omega in [0, 1]               weight of the gain of turning a streaming head into a retrieval head
 * Writes h_layer_is_retrieval [n_layers] (1 = retrieval layer): the choice of p streaming layers
 * that minimises Eq. 5's sum over heads of  alpha (retrieval head made streaming), -omega * alpha
 * (streaming head made retrieval), 0 (kept).  Equal costs: the lower layer index becomes streaming.
 * Optional outputs (may be NULL): h_head_is_retrieval [n_layers * n_heads], the quantile split;
 * *h_cost, the minimum.  Returns ZZ_ERR_INVALID_ARG on NULL / out-of-range / non-finite input. */
int zz_layer_mask_solve(const float* h_alpha, int32_t n_layers, int32_t n_heads, int32_t n_streaming_layers,
                        double omega, uint8_t* h_layer_is_retrieval, uint8_t* h_head_is_retrieval,
                        double* h_cost);

/* Number of kernels this library has launched since it was loaded (all handles). */
int64_t zz_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ZIGZAG_H_ */
