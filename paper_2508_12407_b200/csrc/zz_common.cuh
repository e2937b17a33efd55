// Shared declarations of the CUDA path: parameter blocks passed from the host
// dispatcher to the kernels, and small device helpers.  sm_100a only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "zigzag.h"

namespace zz {

constexpr int kD = 128;            // the usual head_dim (64 is supported by the bf16 kernels; FP8 and paged stores need 128)
constexpr int kRowBytes = kD * 2;  // one K or V row of one head at head_dim 128

// Where the stores of one (layer, sequence) live in the arena, in bf16 elements from the
// arena base.  Index [ZZ_KIND_STREAMING] is the ring group, [ZZ_KIND_RETRIEVAL] the
// append-only group; each group is laid out [head_in_group][slot][128].
//
// Paged retrieval stores (a cache built with a page pool): a page holds 128 tokens of one KV
// head, its K rows [128][128] followed by its V rows.  k_off[ZZ_KIND_RETRIEVAL] is then the
// pool's first K row, v_off[...] the first V row (128 rows further), and the page of token t of
// head h is page_table[tbl + (t / 128) * n_retrieval_heads + h].
struct SeqDesc {
    long long k_off[2];
    long long v_off[2];
    int cap;   // slots per head of the retrieval group (capacity of this sequence)
    int tbl;   // paged stores: first page-table entry of this (layer, sequence)
};

// Split limits of the decode kernel: the last CTA of a (sequence, head) merges the splits with the
// per-split statistics held in rows of kDecodeSplitSlots floats of shared memory, the last slot of a
// row being reserved for the reciprocal of the merged sum.  Host plans never exceed kDecodeMaxSplits.
constexpr int kDecodeSplitSlots = 128;
constexpr int kDecodeMaxSplits = 120;
static_assert(kDecodeMaxSplits < kDecodeSplitSlots, "the merge keeps one spare slot per row");

// FP8 retrieval stores (a cache built with retrieval_kv_fp8): the group of one (layer, sequence)
// holds, from k_off[ZZ_KIND_RETRIEVAL] (counted in 2-byte units like every offset): the K codes
// [head][cap][128] bytes (E4M3), at v_off[...] the V codes likewise, then the K scale bytes
// [head][cap16] and the V scale bytes [head][cap16], cap16 = cap rounded up to 16 (a scale byte e
// stands for 2^(e - 127); one per token and head).
__host__ __device__ inline int fp8_cap16(int cap) { return (cap + 15) & ~15; }
__host__ __device__ inline long long fp8_kscale_byte_off(long long v_off, int n_heads, int cap) {
    return 2 * v_off + (long long)n_heads * cap * kD;
}

constexpr int kPageTokens = 128;
constexpr long long kPageElems = 2LL * kPageTokens * kD;   // K block, then V block

// Page-table writes of one launch (passed by value: no host buffer has to outlive the call).
struct TableUpdate {
    int n;
    int idx[480];
    int val[480];
};

struct AppendParams {
    __nv_bfloat16* arena;
    const SeqDesc* desc;     // [B] of this layer
    int* len;                // [B] of this layer (device lengths)
    int* pos;                // [B][ring] of this layer
    unsigned int* counter;   // blocks-done counter (0 between launches)
    const __nv_bfloat16* k_new;  // [sum n_new][Hkv][128]
    const __nv_bfloat16* v_new;
    const int* head_list;    // [Hkv] source KV heads: first nR retrieval heads, then streaming
    const int* page_table;   // nullptr: contiguous retrieval stores
    int nR, Hkv, ring, S, W, B;
    int D;                   // head_dim (64 or 128)
    int skip_retrieval;      // the retrieval heads' rows were stored by another launch (FP8 stores)
    int n_new[ZZ_MAX_BATCH];
    int tok_off[ZZ_MAX_BATCH];
};

struct DecodeParams {
    __nv_bfloat16* arena;
    int* len;                // [B] device lengths of this layer
    const __nv_bfloat16* q;  // row of sequence b, head h at q + b*q_tok_stride + (q_head0 + h)*128
    __nv_bfloat16* out;      // same addressing as q
    long long q_tok_stride;  // elements between consecutive sequences' rows (n_q_heads * 128)
    int q_head0;             // first query head of this group inside a row
    float* part_o;           // [work item][G][128] split partials of this launch
    float* part_ml;          // [work item][G][2]
    unsigned int* counters;  // [B*Hg], 0 between launches
    int* status;
    int kind;                // which group of the layer
    int ring;                // S+W
    int D;                   // head_dim (selects the kernel instantiation)
    int Hg, G, B;
    int max_splits;          // most splits any sequence of this launch has (<= kDecodeMaxSplits); the kernel
                             // refuses a plan beyond it instead of overrunning its merge rows
    float scale_log2;        // softmax_scale * log2(e)
    // fused append (k_new != nullptr): the token at position len is taken from k_new/v_new
    // ([B][n_kv_total][128], model head order), written to its slot, and attended to
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    const int* head_list;    // [n_kv_total] group-ordered source KV heads
    int* pos;                // [B][ring] ring positions of this layer
    unsigned int* seq_counters;  // [B], 0 between launches
    int kv_head0;            // first entry of head_list that belongs to the group
    int n_kv_total;
    int S, W;
    int bump_len;            // this launch advances len (the last launch of a layer does)
    int appended;            // FP8 stores: the step's token was stored by the launch before this one (the
                             // device length does not count it yet): attend over len + 1 rows
    int gdc_wait;            // 1: wait for the previous launch before touching workspace and output;
                             // 2: wait at kernel entry; 0: never
    int split_start[ZZ_MAX_BATCH + 1];  // prefix sum of per-sequence split counts
    int chunk[ZZ_MAX_BATCH];            // tokens per split of each sequence
    int early_len[ZZ_MAX_BATCH];        // rows of each sequence's retrieval store that were complete before the
                                        // previous launch in the stream began (0: none known): a launch that
                                        // waits at entry may fetch blocks below this length before it waits
    SeqDesc sd[ZZ_MAX_BATCH];           // store addresses of every sequence of this layer
    // several layers in one launch (blockIdx.y): layer_ids[y] is the layer, every per-layer pointer
    // above is then the layer-0 pointer and advances by these strides (elements) per layer; the
    // store addresses come from desc_table[layer * B + b].  layer_ids == nullptr: one layer.
    const int* layer_ids;
    const SeqDesc* desc_table;
    const int* page_table;   // nullptr: contiguous retrieval stores
    long long st_len, st_pos, st_q, st_kv, st_cnt, st_part;
};

// Quantising append into FP8 retrieval stores: rows of the retrieval heads become E4M3 codes plus a
// scale byte.  One layer and a packed chunk (layer_ids == nullptr: n_new / tok_off per sequence), or
// one token per sequence for several layers at once (layer_ids: k_new / v_new are [layer][B][Hkv][128]).
// Does not change the lengths (the launch that follows does).
struct QuantAppendParams {
    unsigned char* arena;
    const SeqDesc* desc_table;   // [L][B]
    const int* len;              // [L][B] device lengths
    const int* head_list;        // [L][Hkv] group-ordered source KV heads (retrieval heads first)
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    const int* layer_ids;        // nullptr: the single layer `layer`
    int* status;
    int layer, nR, Hkv, B;
    int n_new[ZZ_MAX_BATCH];
    int tok_off[ZZ_MAX_BATCH];
};

// FP8 rows [0, len) of one layer's retrieval stores -> bf16 rows in a scratch region laid out like a
// bf16 retrieval group (what the prefill kernel reads when a chunk attends to an FP8 store).
struct DequantParams {
    unsigned char* arena;
    const SeqDesc* src;          // [B] of the layer
    const SeqDesc* dst;          // [B] scratch layout
    const int* len;              // [B]
    int nR, B;
};

struct GatherParams {
    // copies rows of heads between the model's head order and the two compact group buffers
    const __nv_bfloat16* src;
    __nv_bfloat16* dst;
    const int* head_list;    // [Hkv] group-ordered KV heads
    int Hkv, G;
    int D;                   // head_dim
    long long tokens;
    int to_compact;          // 1: model order -> compact (gather); 0: compact -> model order (scatter)
    // several layers in one launch (decode step): token t belongs to layer layer_ids[t / toks_per_layer];
    // src, dst and head_list are then the layer-0 pointers, each layer `toks_per_layer` tokens further
    const int* layer_ids;    // nullptr: one layer
    int toks_per_layer;
};

struct PrefillParams {
    const SeqDesc* desc;     // [B] of this layer
    const int* len;          // [B] device lengths (tokens already in the store)
    const int* pos;          // [B][ring] ring positions of this layer (not read: which token a slot holds follows from len)
    __nv_bfloat16* out;      // row of packed token i, head h at out + i*tok_stride + (q_head0+h)*128
    long long tok_stride;    // n_q_heads * 128
    const int* page_table;   // nullptr: contiguous retrieval stores
    const int* head_list;    // [Hkv] group-ordered source KV heads (for the chunk K/V)
    int* status;
    int kind;                // group served by this launch
    int kv_head0;            // first entry of head_list that belongs to the group
    int q_head0;             // first query head of the group inside a q/out row
    int n_kv_total;          // KV heads per row of the chunk K/V
    int ring, S, W, Hg, G, B;
    int D;                   // head_dim (selects the kernel instantiation)
    int total_tiles;         // 128-row query tiles over the whole batch
    int n_items;             // work items of the launch (set by the launcher)
    float scale_log2;
    int n_new[ZZ_MAX_BATCH];
    int tok_off[ZZ_MAX_BATCH];
    int tile_start[ZZ_MAX_BATCH + 1];
};

// ---- launchers (defined in the .cu files) -------------------------------------------
cudaError_t launch_append(const AppendParams& p, int grid_x, cudaStream_t s);
cudaError_t launch_decode(const DecodeParams& p, int n_items, int warps, cudaStream_t s, int overlap = 0, int n_layers = 1);
cudaError_t launch_regroup(const GatherParams& p, cudaStream_t s, int programmatic);
cudaError_t launch_quant_append(const QuantAppendParams& p, int max_new, int n_layers, cudaStream_t s);
cudaError_t launch_dequant(const DequantParams& p, int max_len, cudaStream_t s);
cudaError_t launch_decode_fp8(const DecodeParams& p, int n_items, int warps, cudaStream_t s, int overlap = 0, int n_layers = 1);
cudaError_t decode_fp8_setup();
cudaError_t launch_reset(int* len, int* pos, int L, int B, int ring, int seq, cudaStream_t s);
cudaError_t launch_table_update(int* table, const TableUpdate& u, cudaStream_t s);
cudaError_t decode_setup();
cudaError_t prefill_setup();
// tensor maps: q [tokens][heads][128] (3-D), chunk k and v [tokens][kv heads][128] (3-D), and the
// arena seen as rows of 128 bf16 (2-D); opaque 128-byte CUtensorMap objects
cudaError_t launch_prefill(const PrefillParams& p, const void* tmap_q, const void* tmap_k,
                           const void* tmap_v, const void* tmap_arena, int n_items, cudaStream_t s);

cudaError_t launch_wait_probe(int* status, unsigned int polls, int* gave_up, cudaStream_t s);

void count_launch(int n = 1);

// Lightweight tracer: when enabled, every launch is bracketed by two CUDA events on its
// stream and accumulated per kernel class.
enum ProfKind { kProfAppend = 0, kProfDecodeR = 1, kProfDecodeS = 2, kProfPrefillR = 3, kProfPrefillS = 4,
                kProfRegroup = 5, kProfOther = 6, kProfKinds = 7 };
void prof_begin(int kind, cudaStream_t s);
void prof_end(int kind, cudaStream_t s);

}  // namespace zz
