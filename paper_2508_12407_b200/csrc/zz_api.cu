// C ABI of the library: handle, layout, validation and per-layer dispatch.
// Every step of the hot path runs in the kernels of the sibling .cu files; this file only
// checks arguments, plans launches and tracks lengths.
#include <cuda.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "zz_common.cuh"

namespace zz {
static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// ---- tracer ------------------------------------------------------------------------------
namespace {
struct ProfRecord { int kind; cudaEvent_t e0, e1; };
struct Profiler {
    int period = 0;                  // 0 = off, n = sample every n-th launch of a class
    long long seen[kProfKinds] = {0};
    std::vector<ProfRecord> recs;
    std::vector<cudaEvent_t> pool;   // events ready for reuse
    cudaEvent_t pending = nullptr;
    cudaEvent_t take() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
        return e;
    }
} g_prof;
}  // namespace
void prof_begin(int kind, cudaStream_t s) {
    g_prof.pending = nullptr;
    if (g_prof.period <= 0) return;
    if ((g_prof.seen[kind]++ % g_prof.period) != 0) return;
    g_prof.pending = g_prof.take();
    if (g_prof.pending) cudaEventRecord(g_prof.pending, s);
}
void prof_end(int kind, cudaStream_t s) {
    if (!g_prof.pending) return;
    cudaEvent_t e1 = g_prof.take();
    if (!e1) { g_prof.pool.push_back(g_prof.pending); g_prof.pending = nullptr; return; }
    cudaEventRecord(e1, s);
    g_prof.recs.push_back(ProfRecord{kind, g_prof.pending, e1});
    g_prof.pending = nullptr;
}
}  // namespace zz

using zz::kD;
using zz::SeqDesc;

namespace {

constexpr int kMaxSplits = zz::kDecodeMaxSplits;   // the decode kernel keeps per-split factors in 128-entry rows
constexpr int kMaxSlots = 512;    // upper bound of CTAs a long-store decode plan may use (2 or 3 per SM)
constexpr size_t kAlign = 256;

size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

struct Layout {
    // workspace sections (byte offsets)
    size_t off_status, off_len, off_pos, off_desc, off_heads, off_counters, off_part_ml, off_part_o,
        off_qc, off_oc, off_dqc, off_doc, off_layer_ids, off_table, work_bytes;
    size_t arena_bytes, counters_per_layer, items_per_layer;
    long long table_entries;   // page-table entries (0: contiguous retrieval stores)
    size_t off_desc_scratch;   // FP8 stores: [L][B] descriptors of the bf16 scratch the prefill kernel reads
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [rows][heads][D] bf16 seen as a 3-D tensor; a box is 128 rows x 1 head x 64 columns (128-byte swizzle)
bool encode_rows3d(CUtensorMap* m, const void* base, long long rows, int heads, int D) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)heads * D * 2};
    cuuint32_t box[3] = {64, 1, 128};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// the arena as [rows][D] bf16; a box is 128 rows x 64 columns
bool encode_rows2d(CUtensorMap* m, const void* base, long long rows, int D) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct zz_cache {
    int L, B, Hq, Hkv, G, D, S, W, ring, max_new;
    float scale;
    std::vector<uint8_t> kind;        // [L*Hkv]
    std::vector<int> nR;              // [L] retrieval KV heads of the layer
    std::vector<int> heads;           // [L*Hkv] group-ordered KV heads (retrieval first), ascending in each group
    std::vector<int> cap;             // [B]
    std::vector<int> len;             // [L*B] host mirror
    std::vector<SeqDesc> desc;        // [L*B]
    std::vector<SeqDesc> desc_scratch;  // [L*B] FP8 caches: the layer's retrieval group in the bf16 scratch
    std::vector<int> layer_ids;       // exclusive retrieval layers (ascending), exclusive streaming, mixed
    int n_excl_R, n_excl_S, n_mixed;
    bool mixed_same_nR;               // every mixed layer has the same number of retrieval heads
    Layout lay;
    unsigned char* arena;
    unsigned char* work;
    int num_sms;
    int decode_min_chunk;
    int decode_short_tokens;
    int decode_overlap;
    int decode_multi_waves;
    bool last_nowait;   // the last launch did not wait for its predecessor: the next one must be an ordinary launch
    int fresh_layer;    // layer whose store rows below the host length the last launch may still be writing
                        // (-1: none, -2: any): no launch fetches them before it has waited for that launch
    bool has_mixed;
    // paged retrieval stores
    bool fp8;                         // retrieval stores hold E4M3 codes + a scale byte per token and head
    bool paged;
    int pool_pages;
    std::vector<int> free_pages;      // stack of free page ids
    std::vector<int> h_table;         // host mirror of the page table
    std::vector<int> pages_of;        // [L*B] token blocks that already have pages
    bool table_dirty;                 // page-table writes were launched: the next decode launch is an ordinary one
    alignas(64) CUtensorMap tmap_arena;
    bool have_tmap_arena;

    int* d_status() const { return reinterpret_cast<int*>(work + lay.off_status); }
    unsigned int* d_append_counter() const { return reinterpret_cast<unsigned int*>(work + lay.off_status + 64); }
    int* d_len(int l) const { return reinterpret_cast<int*>(work + lay.off_len) + (size_t)l * B; }
    int* d_pos(int l) const { return reinterpret_cast<int*>(work + lay.off_pos) + (size_t)l * B * ring; }
    SeqDesc* d_desc(int l) const { return reinterpret_cast<SeqDesc*>(work + lay.off_desc) + (size_t)l * B; }
    SeqDesc* d_desc_scratch(int l) const { return reinterpret_cast<SeqDesc*>(work + lay.off_desc_scratch) + (size_t)l * B; }
    int* d_layer_ids() const { return reinterpret_cast<int*>(work + lay.off_layer_ids); }
    int* d_table() const { return reinterpret_cast<int*>(work + lay.off_table); }
    int* d_heads(int l) const { return reinterpret_cast<int*>(work + lay.off_heads) + (size_t)l * Hkv; }
    unsigned int* d_counters(int l) const {
        return reinterpret_cast<unsigned int*>(work + lay.off_counters) + (size_t)l * lay.counters_per_layer;
    }
    float* d_part_ml(int l) const {
        return reinterpret_cast<float*>(work + lay.off_part_ml) + (size_t)l * lay.items_per_layer * G * 2;
    }
    float* d_part_o(int l) const {
        return reinterpret_cast<float*>(work + lay.off_part_o) + (size_t)l * lay.items_per_layer * G * D;
    }
    __nv_bfloat16* d_qc() const { return reinterpret_cast<__nv_bfloat16*>(work + lay.off_qc); }
    __nv_bfloat16* d_oc() const { return reinterpret_cast<__nv_bfloat16*>(work + lay.off_oc); }
    // compact-order q and out of a decode step over all layers: [L][B][Hq][128]
    __nv_bfloat16* d_dqc() const { return reinterpret_cast<__nv_bfloat16*>(work + lay.off_dqc); }
    __nv_bfloat16* d_doc() const { return reinterpret_cast<__nv_bfloat16*>(work + lay.off_doc); }
    __nv_bfloat16* d_arena() const { return reinterpret_cast<__nv_bfloat16*>(arena); }
    bool mixed(int l) const { return nR[l] > 0 && nR[l] < Hkv; }
};

namespace {

int validate(const zz_config_t* c) {
    if (!c || !c->layer_is_retrieval || !c->capacity) return ZZ_ERR_INVALID_ARG;
    if (c->n_layers < 1 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1) return ZZ_ERR_INVALID_ARG;
    if (c->sink < 0 || c->recent < 1) return ZZ_ERR_INVALID_ARG;
    if (c->max_new_tokens < c->batch) return ZZ_ERR_INVALID_ARG;
    if (!(c->softmax_scale > 0.f)) return ZZ_ERR_INVALID_ARG;
    if (c->head_dim != 128 && c->head_dim != 64) return ZZ_ERR_UNSUPPORTED;
    if (c->head_dim != kD && c->retrieval_kv_fp8) return ZZ_ERR_UNSUPPORTED;      // FP8 stores: head_dim 128 only
    if (c->batch > ZZ_MAX_BATCH) return ZZ_ERR_UNSUPPORTED;
    if (c->n_q_heads % c->n_kv_heads != 0) return ZZ_ERR_UNSUPPORTED;
    if (c->n_q_heads / c->n_kv_heads > 16) return ZZ_ERR_UNSUPPORTED;
    if (c->retrieval_kv_fp8 != 0 && c->retrieval_kv_fp8 != 1) return ZZ_ERR_INVALID_ARG;
    for (int b = 0; b < c->batch; ++b)
        if (c->capacity[b] < 1) return ZZ_ERR_INVALID_ARG;
    return ZZ_OK;
}

uint8_t kind_of(const zz_config_t* c, int l, int h) {
    if (c->kvhead_is_retrieval) return c->kvhead_is_retrieval[(size_t)l * c->n_kv_heads + h] ? 1 : 0;
    return c->layer_is_retrieval[l] ? 1 : 0;
}

// Arena: for each layer, for each sequence: retrieval group K [nR][cap][128], V likewise, then
// streaming group K [nS][S+W][128], V likewise.  Fills `desc` if given.
void compute_layout(const zz_config_t* c, Layout* lay, std::vector<SeqDesc>* desc, long long pool_pages = 0,
                    std::vector<SeqDesc>* desc_scratch = nullptr) {
    const int L = c->n_layers, B = c->batch, Hkv = c->n_kv_heads, Hq = c->n_q_heads;
    const int ring = c->sink + c->recent;
    const int G = Hq / Hkv;
    const int Dh = c->head_dim;     // (FP8 stores exist at head_dim 128 only, where Dh == Dh)
    long long off = 0;  // elements
    long long tbl = 0;  // page-table entries
    const bool paged = pool_pages > 0;
    const bool fp8 = c->retrieval_kv_fp8 != 0;
    bool has_mixed = false;
    int max_nR = 0;
    if (desc) desc->assign((size_t)L * B, SeqDesc());
    for (int l = 0; l < L; ++l) {
        int nR = 0;
        for (int h = 0; h < Hkv; ++h) nR += kind_of(c, l, h);
        const int nS = Hkv - nR;
        if (nR > 0 && nS > 0) has_mixed = true;
        if (nR > max_nR) max_nR = nR;
        for (int b = 0; b < B; ++b) {
            SeqDesc d;
            d.cap = c->capacity[b];
            d.tbl = (int)tbl;
            if (paged) {
                // retrieval rows live in the pool (offsets filled in below): entries [token block][head]
                tbl += (long long)((d.cap + zz::kPageTokens - 1) / zz::kPageTokens) * nR;
                d.k_off[ZZ_KIND_RETRIEVAL] = d.v_off[ZZ_KIND_RETRIEVAL] = 0;
            } else if (fp8) {
                // codes are one byte each (offsets count 2-byte units); the scale bytes follow the V codes
                d.k_off[ZZ_KIND_RETRIEVAL] = off;
                off += (long long)nR * d.cap * Dh / 2;
                d.v_off[ZZ_KIND_RETRIEVAL] = off;
                off += (long long)nR * d.cap * Dh / 2;
                off += (long long)nR * zz::fp8_cap16(d.cap);       // K and V scale bytes: 2 * nR * cap16 bytes
                off = (off + Dh - 1) / Dh * Dh;                     // what follows starts on a whole bf16 row again
                                                                    // (the prefill kernel addresses the arena by rows)
            } else {
                d.k_off[ZZ_KIND_RETRIEVAL] = off;
                off += (long long)nR * d.cap * Dh;
                d.v_off[ZZ_KIND_RETRIEVAL] = off;
                off += (long long)nR * d.cap * Dh;
            }
            d.k_off[ZZ_KIND_STREAMING] = off;
            off += (long long)nS * ring * Dh;
            d.v_off[ZZ_KIND_STREAMING] = off;
            off += (long long)nS * ring * Dh;
            if (desc) (*desc)[(size_t)l * B + b] = d;
        }
    }
    if (paged) {
        // the pool follows the rings; every descriptor points at it
        const long long pool_off = off;
        off += pool_pages * zz::kPageElems;
        if (desc)
            for (auto& d : *desc) {
                d.k_off[ZZ_KIND_RETRIEVAL] = pool_off;
                d.v_off[ZZ_KIND_RETRIEVAL] = pool_off + (long long)zz::kPageTokens * Dh;
            }
    }
    if (fp8) {
        // bf16 scratch for one layer's retrieval rows (K then V per sequence), read by the prefill kernel
        // when a chunk attends to rows already stored; laid out like a bf16 retrieval group
        if (desc_scratch) desc_scratch->assign((size_t)L * B, SeqDesc());
        long long so = off;
        for (int b = 0; b < B; ++b) {
            for (int l = 0; l < L && desc_scratch; ++l) {
                int nR = 0;
                for (int h = 0; h < Hkv; ++h) nR += kind_of(c, l, h);
                SeqDesc d = (*desc)[(size_t)l * B + b];
                d.k_off[ZZ_KIND_RETRIEVAL] = so;
                d.v_off[ZZ_KIND_RETRIEVAL] = so + (long long)nR * d.cap * Dh;
                (*desc_scratch)[(size_t)l * B + b] = d;
            }
            so += 2LL * max_nR * c->capacity[b] * Dh;
        }
        off = so;
    }
    lay->table_entries = paged ? tbl : 0;
    // one spare tile of rows so that a 128-row tile read starting at the last valid row of the
    // last store stays inside the tensor map's extent (out-of-extent rows read as zero anyway)
    lay->arena_bytes = align_up((size_t)off * 2 + 128 * Dh * 2);
    size_t w = 0;
    lay->off_status = w; w += kAlign;
    lay->off_len = w; w += align_up((size_t)L * B * sizeof(int));
    lay->off_pos = w; w += align_up((size_t)L * B * ring * sizeof(int));
    lay->off_desc = w; w += align_up((size_t)L * B * sizeof(SeqDesc));
    lay->off_heads = w; w += align_up((size_t)L * Hkv * sizeof(int));
    lay->off_layer_ids = w; w += align_up((size_t)L * sizeof(int));
    lay->off_table = w; w += align_up((size_t)lay->table_entries * sizeof(int));
    lay->off_desc_scratch = w;
    if (fp8) w += align_up((size_t)L * B * sizeof(SeqDesc));
    // per layer: arrival counters and the split partials of the layer's launches, indexed by work
    // item (at most kMaxSlots + B * Hkv items per launch), so that the launches of different
    // layers share no scratch and may overlap
    lay->counters_per_layer = (size_t)(B * Hkv + B);
    lay->items_per_layer = (size_t)kMaxSlots + (size_t)B * Hkv;
    lay->off_counters = w; w += align_up((size_t)L * lay->counters_per_layer * sizeof(unsigned int));
    lay->off_part_ml = w; w += align_up((size_t)L * lay->items_per_layer * G * 2 * sizeof(float));
    lay->off_part_o = w; w += align_up((size_t)L * lay->items_per_layer * G * Dh * sizeof(float));
    lay->off_qc = w;
    if (has_mixed) w += align_up((size_t)c->max_new_tokens * Hq * Dh * 2);
    lay->off_oc = w;
    if (has_mixed) w += align_up((size_t)c->max_new_tokens * Hq * Dh * 2);
    lay->off_dqc = w;
    if (has_mixed) w += align_up((size_t)L * B * Hq * Dh * 2);
    lay->off_doc = w;
    if (has_mixed) w += align_up((size_t)L * B * Hq * Dh * 2);
    lay->work_bytes = w;
}

bool bad_layer(const zz_cache* c, int layer) { return !c || layer < 0 || layer >= c->L; }

// Split plan of one decode launch.  Short stores: 8-warp CTAs (one per SM) that each take up to
// 384 tokens, so a warp's chain is at most three dependent steps.  Long stores: 4-warp CTAs
// (ctas_per_sm of them fit an SM), all work items in one wave, every sequence cut into equal splits.
void plan_splits(const zz_cache* c, const int* n, int Hg, int* warps, int* chunk, int* split_start, int n_multi = 1,
                 int ctas_per_sm = 2) {
    long long total = 0;
    for (int b = 0; b < c->B; ++b) total += n[b];
    split_start[0] = 0;
    // the short plan has one split per decode_short_tokens tokens: it serves a launch only if no
    // sequence needs more splits than the kernel's merge can hold (one KV head and ~50K tokens would)
    bool short_ok = c->decode_short_tokens > 0 && total * Hg <= (long long)c->num_sms * c->decode_short_tokens;
    for (int b = 0; b < c->B && short_ok; ++b)
        if ((n[b] + c->decode_short_tokens - 1) / c->decode_short_tokens > kMaxSplits) short_ok = false;
    if (short_ok) {
        *warps = 8;
        for (int b = 0; b < c->B; ++b) {
            int s = (n[b] + c->decode_short_tokens - 1) / c->decode_short_tokens;
            if (s < 1) s = 1;
            chunk[b] = c->decode_short_tokens;
            split_start[b + 1] = split_start[b] + s;
        }
        return;
    }
    *warps = 4;
    int slots = ctas_per_sm * c->num_sms < kMaxSlots ? ctas_per_sm * c->num_sms : kMaxSlots;
    // a grid over several layers fills the GPU with all of them together: each layer is cut into
    // fewer, longer items (decode_multi_waves waves of CTAs over the whole grid), which spends less
    // on per-CTA ramp-up, merge and partials
    if (n_multi > 1) {
        int s = (int)(((long long)slots * c->decode_multi_waves + n_multi - 1) / n_multi);
        const int floor_items = 4 * c->B * Hg;        // keep several splits per sequence for ragged batches
        if (s < floor_items) s = floor_items;
        if (s < slots) slots = s;
    }
    long long per = (total * Hg + slots - 1) / slots;   // tokens per work item if all were equal
    if (per < c->decode_min_chunk) per = c->decode_min_chunk;
    for (;;) {
        long long items = 0;
        int worst = 0;
        for (int b = 0; b < c->B; ++b) {
            const int s = (int)((n[b] + per - 1) / per);
            items += (long long)(s > 0 ? s : 1) * Hg;
            if (s > worst) worst = s;
        }
        if ((items <= slots || per >= total) && worst <= kMaxSplits) break;
        per += 16;
    }
    for (int b = 0; b < c->B; ++b) {
        int s = (int)((n[b] + per - 1) / per);
        if (s < 1) s = 1;
        chunk[b] = (n[b] + s - 1) / s;            // equal splits inside the sequence
        if (chunk[b] < 1) chunk[b] = 1;
        if (c->paged || c->fp8) {
            // splits start at multiples of 16 tokens, so that no 16-token block straddles a page (and the
            // scale bytes of a block of an FP8 store are one aligned 16-byte piece)
            chunk[b] = (chunk[b] + 15) / 16 * 16;
            s = (n[b] + chunk[b] - 1) / chunk[b];
            if (s < 1) s = 1;
        }
        split_start[b + 1] = split_start[b] + s;
    }
}

// Paged stores: make sure that layers [l0, l1) have pages for `add[b]` more tokens per sequence.
// All or nothing: when the pool cannot cover the request nothing is taken and nothing is launched.
// The new table entries reach the device through small kernels on the caller's stream (values
// passed by value), so they are ordered before the launches that follow and no host buffer has to
// stay untouched afterwards.
int reserve_pages(zz_cache* c, int l0, int l1, const int32_t* add, cudaStream_t st) {
    if (!c->paged) return ZZ_OK;
    long long need = 0;
    for (int l = l0; l < l1; ++l) {
        if (c->nR[l] == 0) continue;
        for (int b = 0; b < c->B; ++b) {
            const long long nl = (long long)c->len[(size_t)l * c->B + b] + add[b];
            const long long blocks = (nl + zz::kPageTokens - 1) / zz::kPageTokens - c->pages_of[(size_t)l * c->B + b];
            if (blocks > 0) need += blocks * c->nR[l];
        }
    }
    if (need == 0) return ZZ_OK;
    if (need > (long long)c->free_pages.size()) return ZZ_ERR_CAPACITY;
    zz::TableUpdate u;
    u.n = 0;
    auto flush = [&]() -> bool {
        if (u.n == 0) return true;
        const bool ok = zz::launch_table_update(c->d_table(), u, st) == cudaSuccess;
        u.n = 0;
        return ok;
    };
    for (int l = l0; l < l1; ++l) {
        const int nR = c->nR[l];
        if (nR == 0) continue;
        for (int b = 0; b < c->B; ++b) {
            const size_t lb = (size_t)l * c->B + b;
            const long long nl = (long long)c->len[lb] + add[b];
            const int want = (int)((nl + zz::kPageTokens - 1) / zz::kPageTokens);
            for (int g = c->pages_of[lb]; g < want; ++g)
                for (int h = 0; h < nR; ++h) {
                    const int page = c->free_pages.back();
                    c->free_pages.pop_back();
                    const int idx = c->desc[lb].tbl + g * nR + h;
                    c->h_table[idx] = page;
                    u.idx[u.n] = idx;
                    u.val[u.n] = page;
                    if (++u.n == 480 && !flush()) return ZZ_ERR_CUDA;
                }
            if (want > c->pages_of[lb]) c->pages_of[lb] = want;
        }
    }
    if (!flush()) return ZZ_ERR_CUDA;
    c->table_dirty = true;
    c->last_nowait = false;   // the table writes were ordinary launches
    c->fresh_layer = -2;
    return ZZ_OK;
}

// k_new/v_new != nullptr: fused append of one token per sequence (host lengths not yet bumped)
int launch_decode_group(zz_cache* c, int layer, int kind, const __nv_bfloat16* q, __nv_bfloat16* out,
                        int q_head0, cudaStream_t st, const __nv_bfloat16* k_new = nullptr,
                        const __nv_bfloat16* v_new = nullptr, int bump_len = 0, int overlap = 0,
                        const int* d_layer_ids = nullptr, int n_multi = 1) {
    const int Hg = (kind == ZZ_KIND_RETRIEVAL) ? c->nR[layer] : c->Hkv - c->nR[layer];
    if (Hg == 0) return ZZ_OK;
    // FP8 retrieval stores: the step's token has been stored by a quantising append launched just
    // before (quant_append_step); the kernel attends over len + 1 rows and fuses nothing
    const bool fp8 = c->fp8 && kind == ZZ_KIND_RETRIEVAL;
    const bool with_token = k_new != nullptr;
    zz::DecodeParams p;
    memset(&p, 0, sizeof p);
    p.arena = c->d_arena();
    p.len = c->d_len(layer);
    for (int b = 0; b < c->B; ++b) p.sd[b] = c->desc[(size_t)layer * c->B + b];
    p.k_new = fp8 ? nullptr : k_new;
    p.v_new = fp8 ? nullptr : v_new;
    p.appended = (fp8 && with_token) ? 1 : 0;
    p.head_list = c->d_heads(layer);
    p.pos = c->d_pos(layer);
    p.seq_counters = c->d_counters(layer) + (size_t)c->B * c->Hkv;
    p.kv_head0 = (kind == ZZ_KIND_RETRIEVAL) ? 0 : c->nR[layer];
    p.n_kv_total = c->Hkv;
    p.S = c->S;
    p.W = c->W;
    p.bump_len = bump_len;
    p.q = q;
    p.out = out;
    p.q_tok_stride = (long long)c->Hq * c->D;
    p.D = c->D;
    p.q_head0 = q_head0;
    p.part_o = c->d_part_o(layer);
    p.part_ml = c->d_part_ml(layer);
    p.counters = c->d_counters(layer);
    p.status = c->d_status();
    p.kind = kind;
    p.ring = c->ring;
    p.Hg = Hg;
    p.G = c->G;
    p.B = c->B;
    p.max_splits = kMaxSplits;
    p.scale_log2 = c->scale * 1.4426950408889634f;
    p.page_table = c->paged ? c->d_table() : nullptr;
    int n[ZZ_MAX_BATCH];
    for (int b = 0; b < c->B; ++b) {
        const int len = c->len[(size_t)layer * c->B + b] + (with_token ? 1 : 0);
        n[b] = (kind == ZZ_KIND_RETRIEVAL) ? len : (len < c->ring ? len : c->ring);
    }
    int warps = 4;
    // (the FP8 kernels' 4-warp CTAs fit three to an SM, the bf16 kernel's two)
    plan_splits(c, n, Hg, &warps, p.chunk, p.split_start, d_layer_ids ? n_multi : 1, fp8 ? 3 : 2);
    const int items = p.split_start[c->B] * Hg;
    const int pk = (kind == ZZ_KIND_RETRIEVAL) ? zz::kProfDecodeR : zz::kProfDecodeS;
    zz::prof_begin(pk, st);
    // A programmatic launch orders itself only against its immediate predecessor.  After a launch
    // that did not wait for its own predecessor, only an ordinary launch (full stream order) or
    // another launch of the same independent chain may follow.
    if (c->last_nowait && overlap != 2) overlap = 0;
    // page-table writes precede this launch as ordinary launches: read them in full stream order
    if (c->table_dirty) overlap = 0;
    c->table_dirty = false;
    c->last_nowait = (overlap == 2);
    // Rows a launch may fetch before it waits for its predecessor: those of a contiguous retrieval
    // store that were complete before the predecessor began.  The host length counts them, unless the
    // predecessor itself appended to this layer.
    const bool early = overlap == 3 && kind == ZZ_KIND_RETRIEVAL && !fp8 && !c->paged && !d_layer_ids &&
                       (c->fresh_layer == -1 || (c->fresh_layer >= 0 && c->fresh_layer != layer));
    for (int b = 0; b < c->B; ++b) p.early_len[b] = early ? c->len[(size_t)layer * c->B + b] : 0;
    // what this launch leaves behind for the next one: a launch that does not wait at entry may still
    // run beside its own predecessor, so nothing is known to be complete after it
    if (overlap == 1 || overlap == 2 || d_layer_ids) c->fresh_layer = -2;
    else if (with_token) c->fresh_layer = layer;
    else c->fresh_layer = -1;
    if (d_layer_ids) {
        // one launch for n_multi layers with identical lengths: `layer` stands for all of them in the
        // plan above; every per-layer pointer becomes the layer-0 pointer plus a stride per layer
        p.layer_ids = d_layer_ids;
        p.desc_table = c->d_desc(0);
        p.len = c->d_len(0);
        p.pos = c->d_pos(0);
        p.head_list = c->d_heads(0);
        p.counters = c->d_counters(0);
        p.seq_counters = c->d_counters(0) + (size_t)c->B * c->Hkv;
        p.part_o = c->d_part_o(0);
        p.part_ml = c->d_part_ml(0);
        p.st_len = c->B;
        p.st_pos = (long long)c->B * c->ring;
        p.st_q = (long long)c->B * c->Hq * c->D;
        p.st_kv = (long long)c->B * c->Hkv * c->D;
        p.st_cnt = (long long)c->lay.counters_per_layer;
        p.st_part = (long long)c->lay.items_per_layer * c->G;
    }
    const cudaError_t e = fp8 ? zz::launch_decode_fp8(p, items, warps, st, overlap, n_multi)
                              : zz::launch_decode(p, items, warps, st, overlap, n_multi);
    zz::prof_end(pk, st);
    return e == cudaSuccess ? ZZ_OK : ZZ_ERR_CUDA;
}

// FP8 caches: store (quantised) the rows a call adds to the retrieval heads.  Chunk form: one layer,
// n_new[b] packed tokens per sequence.  Step form (n_new == nullptr): one token per sequence for
// `n_layers` layers listed in d_layer_ids, k/v being [layer][B][Hkv][128]; the layers must have the
// same number of retrieval heads.  The lengths stay as they are (the launch after this one moves them).
int quant_append(zz_cache* c, int layer, const __nv_bfloat16* k, const __nv_bfloat16* v, const int32_t* n_new,
                 const int* d_layer_ids, int n_layers, cudaStream_t st) {
    const int nR = c->nR[layer];
    if (nR == 0) return ZZ_OK;
    zz::QuantAppendParams p;
    memset(&p, 0, sizeof p);
    p.arena = c->arena;
    p.desc_table = c->d_desc(0);
    p.len = c->d_len(0);
    p.head_list = c->d_heads(0);
    p.k_new = k;
    p.v_new = v;
    p.layer_ids = d_layer_ids;
    p.status = c->d_status();
    p.layer = layer;
    p.nR = nR;
    p.Hkv = c->Hkv;
    p.B = c->B;
    int off = 0, worst = 1;
    for (int b = 0; b < c->B; ++b) {
        p.n_new[b] = n_new ? n_new[b] : 1;
        p.tok_off[b] = off;
        off += p.n_new[b];
        if (p.n_new[b] > worst) worst = p.n_new[b];
    }
    zz::prof_begin(zz::kProfAppend, st);
    c->last_nowait = false;
    c->fresh_layer = d_layer_ids ? -2 : layer;
    const cudaError_t e = zz::launch_quant_append(p, worst, d_layer_ids ? n_layers : 1, st);
    zz::prof_end(zz::kProfAppend, st);
    return e == cudaSuccess ? ZZ_OK : ZZ_ERR_CUDA;
}

int regroup(zz_cache* c, int layer, const __nv_bfloat16* src, __nv_bfloat16* dst, long long tokens,
            int to_compact, cudaStream_t st) {
    zz::GatherParams g;
    g.src = src;
    g.dst = dst;
    g.head_list = c->d_heads(layer < 0 ? 0 : layer);
    g.Hkv = c->Hkv;
    g.G = c->G;
    g.D = c->D;
    g.tokens = tokens;
    g.to_compact = to_compact;
    g.layer_ids = nullptr;
    g.toks_per_layer = 0;
    if (layer < 0) {
        // every mixed layer of a decode step at once (tokens = n_mixed * B)
        g.head_list = c->d_heads(0);
        g.layer_ids = c->d_layer_ids() + c->n_excl_R + c->n_excl_S;
        g.toks_per_layer = c->B;
    }
    zz::prof_begin(zz::kProfRegroup, st);
    const cudaError_t e = zz::launch_regroup(g, st, c->last_nowait ? 0 : 1);
    c->last_nowait = false;
    c->fresh_layer = -2;     // (the regroup launch may itself run beside its predecessor)
    zz::prof_end(zz::kProfRegroup, st);
    return e == cudaSuccess ? ZZ_OK : ZZ_ERR_CUDA;
}

int launch_prefill_group(zz_cache* c, int layer, int kind, const CUtensorMap* tq, const CUtensorMap* tk,
                         const CUtensorMap* tv, __nv_bfloat16* out, int q_head0, const int32_t* n_new,
                         cudaStream_t st) {
    const int nR = c->nR[layer];
    const int Hg = (kind == ZZ_KIND_RETRIEVAL) ? nR : c->Hkv - nR;
    if (Hg == 0) return ZZ_OK;
    const bool fp8 = c->fp8 && kind == ZZ_KIND_RETRIEVAL;
    if (fp8) {
        // rows already stored are expanded to bf16 in the scratch (exactly: an FP8 value is a bf16
        // number), and the kernel reads them there; the chunk's own K/V are attended to as given
        int max_len = 0;
        for (int b = 0; b < c->B; ++b) max_len = std::max(max_len, c->len[(size_t)layer * c->B + b]);
        if (max_len > 0) {
            zz::DequantParams dq;
            dq.arena = c->arena;
            dq.src = c->d_desc(layer);
            dq.dst = c->d_desc_scratch(layer);
            dq.len = c->d_len(layer);
            dq.nR = nR;
            dq.B = c->B;
            zz::prof_begin(zz::kProfOther, st);
            const cudaError_t de = zz::launch_dequant(dq, max_len, st);
            zz::prof_end(zz::kProfOther, st);
            if (de != cudaSuccess) return ZZ_ERR_CUDA;
        }
    }
    zz::PrefillParams p;
    memset(&p, 0, sizeof p);
    p.desc = fp8 ? c->d_desc_scratch(layer) : c->d_desc(layer);
    p.len = c->d_len(layer);
    p.pos = c->d_pos(layer);
    p.out = out;
    p.tok_stride = (long long)c->Hq * c->D;
    p.D = c->D;
    p.head_list = c->d_heads(layer);
    p.page_table = c->paged ? c->d_table() : nullptr;
    p.status = c->d_status();
    p.kind = kind;
    p.kv_head0 = (kind == ZZ_KIND_RETRIEVAL) ? 0 : nR;
    p.q_head0 = q_head0;
    p.n_kv_total = c->Hkv;
    p.ring = c->ring;
    p.S = c->S;
    p.W = c->W;
    p.Hg = Hg;
    p.G = c->G;
    p.B = c->B;
    p.scale_log2 = c->scale * 1.4426950408889634f;
    int off = 0, tiles = 0;
    for (int b = 0; b < c->B; ++b) {
        p.n_new[b] = n_new[b];
        p.tok_off[b] = off;
        p.tile_start[b] = tiles;
        off += n_new[b];
        tiles += (n_new[b] + 127) / 128;
    }
    p.tile_start[c->B] = tiles;
    p.total_tiles = tiles;
    const int pairs = (c->G + 1) / 2;
    const long long items = (long long)tiles * Hg * pairs;
    if (items == 0) return ZZ_OK;
    if (items > 0x7fffffffLL) return ZZ_ERR_UNSUPPORTED;
    const int pk = (kind == ZZ_KIND_RETRIEVAL) ? zz::kProfPrefillR : zz::kProfPrefillS;
    zz::prof_begin(pk, st);
    c->last_nowait = false;   // an ordinary launch: full stream order
    c->fresh_layer = -1;
    const cudaError_t e = zz::launch_prefill(p, tq, tk, tv, &c->tmap_arena, (int)items, st);
    zz::prof_end(pk, st);
    return e == cudaSuccess ? ZZ_OK : ZZ_ERR_CUDA;
}

}  // namespace

extern "C" {

int zz_version(void) { return 100; }

const char* zz_status_str(int s) {
    switch (s) {
        case ZZ_OK: return "ok";
        case ZZ_ERR_INVALID_ARG: return "invalid argument";
        case ZZ_ERR_UNSUPPORTED: return "unsupported configuration";
        case ZZ_ERR_CAPACITY: return "retrieval store capacity exceeded";
        case ZZ_ERR_WORKSPACE: return "arena or workspace too small";
        case ZZ_ERR_CUDA: return "CUDA error";
        case ZZ_ERR_TIMEOUT: return "bounded device-side wait expired";
        default: return "unknown status";
    }
}

int64_t zz_launch_count(void) { return zz::g_launches.load(std::memory_order_relaxed); }

static int query_impl(const zz_config_t* cfg, long long pool_pages, size_t* arena_bytes, size_t* workspace_bytes) {
    const int v = validate(cfg);
    if (v != ZZ_OK) return v;
    if (!arena_bytes || !workspace_bytes) return ZZ_ERR_INVALID_ARG;
    if (cfg->retrieval_kv_fp8 && pool_pages > 0) return ZZ_ERR_UNSUPPORTED;   // FP8 stores are contiguous
    if (cfg->head_dim != kD && pool_pages > 0) return ZZ_ERR_UNSUPPORTED;     // pages hold rows of 128
    Layout lay;
    compute_layout(cfg, &lay, nullptr, pool_pages);
    if (lay.table_entries > 0x7fffffffLL) return ZZ_ERR_UNSUPPORTED;
    *arena_bytes = lay.arena_bytes;
    *workspace_bytes = lay.work_bytes;
    return ZZ_OK;
}

int zz_cache_query(const zz_config_t* cfg, size_t* arena_bytes, size_t* workspace_bytes) {
    return query_impl(cfg, 0, arena_bytes, workspace_bytes);
}

int zz_cache_query_paged(const zz_config_t* cfg, int32_t pool_pages, size_t* arena_bytes, size_t* workspace_bytes) {
    if (pool_pages < 1) return ZZ_ERR_INVALID_ARG;
    return query_impl(cfg, pool_pages, arena_bytes, workspace_bytes);
}

static int create_impl(const zz_config_t* cfg, long long pool_pages, void* d_arena, size_t arena_bytes,
                       void* d_workspace, size_t workspace_bytes, zz_cache_t** out);

int zz_cache_create(const zz_config_t* cfg, void* d_arena, size_t arena_bytes, void* d_workspace,
                    size_t workspace_bytes, zz_cache_t** out) {
    return create_impl(cfg, 0, d_arena, arena_bytes, d_workspace, workspace_bytes, out);
}

int zz_cache_create_paged(const zz_config_t* cfg, int32_t pool_pages, void* d_arena, size_t arena_bytes,
                          void* d_workspace, size_t workspace_bytes, zz_cache_t** out) {
    if (pool_pages < 1) return ZZ_ERR_INVALID_ARG;
    return create_impl(cfg, pool_pages, d_arena, arena_bytes, d_workspace, workspace_bytes, out);
}

int zz_cache_pages(const zz_cache_t* c, int32_t* total, int32_t* free_now) {
    if (!c || !total || !free_now) return ZZ_ERR_INVALID_ARG;
    *total = c->paged ? c->pool_pages : 0;
    *free_now = c->paged ? (int32_t)c->free_pages.size() : 0;
    return ZZ_OK;
}

static int create_impl(const zz_config_t* cfg, long long pool_pages, void* d_arena, size_t arena_bytes,
                       void* d_workspace, size_t workspace_bytes, zz_cache_t** out) {
    const int v = validate(cfg);
    if (v != ZZ_OK) return v;
    if (!d_arena || !d_workspace || !out) return ZZ_ERR_INVALID_ARG;
    if (cfg->retrieval_kv_fp8 && pool_pages > 0) return ZZ_ERR_UNSUPPORTED;
    if (cfg->head_dim != kD && pool_pages > 0) return ZZ_ERR_UNSUPPORTED;
    if (((uintptr_t)d_arena % kAlign) || ((uintptr_t)d_workspace % kAlign)) return ZZ_ERR_INVALID_ARG;
    zz_cache* c = new (std::nothrow) zz_cache();
    if (!c) return ZZ_ERR_INVALID_ARG;
    c->L = cfg->n_layers; c->B = cfg->batch; c->Hq = cfg->n_q_heads; c->Hkv = cfg->n_kv_heads;
    c->D = cfg->head_dim;
    c->G = c->Hq / c->Hkv; c->S = cfg->sink; c->W = cfg->recent; c->ring = c->S + c->W;
    c->max_new = cfg->max_new_tokens; c->scale = cfg->softmax_scale;
    c->decode_min_chunk = 256;
    c->decode_short_tokens = 384;
    c->decode_overlap = 3;
    c->last_nowait = false;
    c->fresh_layer = -1;
    c->decode_multi_waves = 8;
    c->fp8 = cfg->retrieval_kv_fp8 != 0;
    compute_layout(cfg, &c->lay, &c->desc, pool_pages, &c->desc_scratch);
    if (c->lay.table_entries > 0x7fffffffLL) {
        delete c;
        return ZZ_ERR_UNSUPPORTED;
    }
    if (arena_bytes < c->lay.arena_bytes || workspace_bytes < c->lay.work_bytes) {
        delete c;
        return ZZ_ERR_WORKSPACE;
    }
    c->paged = pool_pages > 0;
    c->pool_pages = (int)pool_pages;
    c->table_dirty = false;
    if (c->paged) {
        c->h_table.assign((size_t)c->lay.table_entries, -1);
        c->pages_of.assign((size_t)c->L * c->B, 0);
        c->free_pages.resize((size_t)pool_pages);
        for (long long i = 0; i < pool_pages; ++i) c->free_pages[(size_t)i] = (int)(pool_pages - 1 - i);  // page 0 on top
    }
    c->arena = static_cast<unsigned char*>(d_arena);
    c->work = static_cast<unsigned char*>(d_workspace);
    c->kind.resize((size_t)c->L * c->Hkv);
    c->nR.assign(c->L, 0);
    c->heads.resize((size_t)c->L * c->Hkv);
    c->has_mixed = false;
    for (int l = 0; l < c->L; ++l) {
        int r = 0;
        for (int h = 0; h < c->Hkv; ++h) {
            c->kind[(size_t)l * c->Hkv + h] = kind_of(cfg, l, h);
            r += c->kind[(size_t)l * c->Hkv + h];
        }
        c->nR[l] = r;
        int ir = 0, is = r;
        for (int h = 0; h < c->Hkv; ++h) {
            if (c->kind[(size_t)l * c->Hkv + h]) c->heads[(size_t)l * c->Hkv + ir++] = h;
            else c->heads[(size_t)l * c->Hkv + is++] = h;
        }
        if (r > 0 && r < c->Hkv) c->has_mixed = true;
    }
    c->n_excl_R = c->n_excl_S = 0;
    for (int l = 0; l < c->L; ++l)
        if (c->nR[l] == c->Hkv) { c->layer_ids.push_back(l); ++c->n_excl_R; }
    for (int l = 0; l < c->L; ++l)
        if (c->nR[l] == 0) { c->layer_ids.push_back(l); ++c->n_excl_S; }
    c->n_mixed = 0;
    c->mixed_same_nR = true;
    for (int l = 0; l < c->L; ++l)
        if (c->mixed(l)) {
            if (c->n_mixed > 0 && c->nR[l] != c->nR[c->layer_ids.back()]) c->mixed_same_nR = false;
            c->layer_ids.push_back(l);
            ++c->n_mixed;
        }
    c->cap.assign(cfg->capacity, cfg->capacity + c->B);
    c->len.assign((size_t)c->L * c->B, 0);

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = zz::decode_setup();
    if (e == cudaSuccess) e = zz::prefill_setup();
    if (e == cudaSuccess && c->fp8) e = zz::decode_fp8_setup();
    if (e == cudaSuccess) e = cudaMemset(c->arena, 0, c->lay.arena_bytes);
    if (e == cudaSuccess) e = cudaMemset(c->work, 0, c->lay.off_part_ml);
    if (e == cudaSuccess) e = cudaMemset(c->work + c->lay.off_pos, 0xff, (size_t)c->L * c->B * c->ring * sizeof(int));
    if (e == cudaSuccess && c->lay.table_entries > 0)     // no page anywhere yet
        e = cudaMemset(c->work + c->lay.off_table, 0xff, (size_t)c->lay.table_entries * sizeof(int));
    if (e == cudaSuccess)
        e = cudaMemcpy(c->work + c->lay.off_desc, c->desc.data(), c->desc.size() * sizeof(SeqDesc),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess && c->fp8)
        e = cudaMemcpy(c->work + c->lay.off_desc_scratch, c->desc_scratch.data(), c->desc_scratch.size() * sizeof(SeqDesc),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(c->work + c->lay.off_heads, c->heads.data(), c->heads.size() * sizeof(int),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(c->work + c->lay.off_layer_ids, c->layer_ids.data(), c->layer_ids.size() * sizeof(int),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        delete c;
        return ZZ_ERR_CUDA;
    }
    c->have_tmap_arena = encode_rows2d(&c->tmap_arena, c->arena, (long long)(c->lay.arena_bytes / (c->D * 2)), c->D);
    *out = c;
    return ZZ_OK;
}

int zz_cache_destroy(zz_cache_t* c) {
    if (!c) return ZZ_ERR_INVALID_ARG;
    delete c;
    return ZZ_OK;
}

int zz_cache_reset(zz_cache_t* c, int seq, void* stream) {
    if (!c || seq < -1 || seq >= c->B) return ZZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c->last_nowait = false;
    c->fresh_layer = -1;
    if (zz::launch_reset(c->d_len(0), c->d_pos(0), c->L, c->B, c->ring, seq, st) != cudaSuccess)
        return ZZ_ERR_CUDA;
    zz::TableUpdate u;
    u.n = 0;
    bool ok = true;
    for (int l = 0; l < c->L; ++l)
        for (int b = 0; b < c->B; ++b)
            if (seq < 0 || seq == b) {
                const size_t lb = (size_t)l * c->B + b;
                c->len[lb] = 0;
                if (c->paged) {
                    // the sequence's pages go back to the pool (work already in the stream that reads
                    // them is ordered before whatever writes them next on the same stream); their
                    // table entries read "no page" again
                    const int n = c->pages_of[lb] * c->nR[l];
                    for (int i = 0; i < n; ++i) {
                        const int idx = c->desc[lb].tbl + i;
                        c->free_pages.push_back(c->h_table[idx]);
                        c->h_table[idx] = -1;
                        u.idx[u.n] = idx;
                        u.val[u.n] = -1;
                        if (++u.n == 480) {
                            ok = ok && zz::launch_table_update(c->d_table(), u, st) == cudaSuccess;
                            u.n = 0;
                        }
                    }
                    c->pages_of[lb] = 0;
                }
            }
    if (u.n > 0) ok = ok && zz::launch_table_update(c->d_table(), u, st) == cudaSuccess;
    return ok ? ZZ_OK : ZZ_ERR_CUDA;
}

int zz_cache_len(const zz_cache_t* c, int layer, int seq, int32_t* len) {
    if (bad_layer(c, layer) || seq < 0 || seq >= c->B || !len) return ZZ_ERR_INVALID_ARG;
    *len = c->len[(size_t)layer * c->B + seq];
    return ZZ_OK;
}

int zz_cache_reserve(zz_cache_t* c, int32_t extra_tokens, void* stream) {
    if (!c || extra_tokens < 0) return ZZ_ERR_INVALID_ARG;
    for (int l = 0; l < c->L; ++l)
        for (int b = 0; b < c->B; ++b) {
            const long long nl = (long long)c->len[(size_t)l * c->B + b] + extra_tokens;
            if (nl > 0x7fffffffLL || (c->nR[l] > 0 && nl > c->cap[b])) return ZZ_ERR_CAPACITY;
        }
    int32_t add[ZZ_MAX_BATCH];
    for (int b = 0; b < c->B; ++b) add[b] = extra_tokens;
    return reserve_pages(c, 0, c->L, add, static_cast<cudaStream_t>(stream));
}

int zz_cache_sync_len(zz_cache_t* c, void* stream) {
    if (!c) return ZZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::vector<int> dev(c->len.size());
    if (cudaMemcpyAsync(dev.data(), c->d_len(0), dev.size() * sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return ZZ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZZ_ERR_CUDA;
    c->len = dev;
    return ZZ_OK;
}

int zz_tune(zz_cache_t* c, const char* key, int value) {
    if (!c || !key) return ZZ_ERR_INVALID_ARG;
    if (!strcmp(key, "decode_min_chunk")) {
        if (value < 16 || value % 16) return ZZ_ERR_INVALID_ARG;
        c->decode_min_chunk = value;
        return ZZ_OK;
    }
    if (!strcmp(key, "decode_multi_waves")) {
        if (value < 1 || value > 64) return ZZ_ERR_INVALID_ARG;
        c->decode_multi_waves = value;
        return ZZ_OK;
    }
    if (!strcmp(key, "decode_overlap")) {
        if (value < 0 || value > 3) return ZZ_ERR_INVALID_ARG;
        c->decode_overlap = value;
        return ZZ_OK;
    }
    if (!strcmp(key, "decode_short_tokens")) {
        if (value < 0 || value % 16) return ZZ_ERR_INVALID_ARG;
        c->decode_short_tokens = value;
        return ZZ_OK;
    }
    return ZZ_ERR_INVALID_ARG;
}

int zz_kv_append(zz_cache_t* c, int layer, const void* d_k, const void* d_v, const int32_t* h_n_new,
                 void* stream) {
    if (bad_layer(c, layer) || !d_k || !d_v || !h_n_new) return ZZ_ERR_INVALID_ARG;
    if (((uintptr_t)d_k | (uintptr_t)d_v) & 15) return ZZ_ERR_INVALID_ARG;
    const int nR = c->nR[layer], nS = c->Hkv - nR;
    long long total = 0, worst = 0;
    for (int b = 0; b < c->B; ++b) {
        if (h_n_new[b] < 0) return ZZ_ERR_INVALID_ARG;
        const long long nl = (long long)c->len[(size_t)layer * c->B + b] + h_n_new[b];
        if (nl > 0x7fffffffLL) return ZZ_ERR_CAPACITY;
        if (nR > 0 && nl > c->cap[b]) return ZZ_ERR_CAPACITY;
        total += h_n_new[b];
    }
    if (total == 0) return ZZ_OK;
    {
        const int rp = reserve_pages(c, layer, layer + 1, h_n_new, static_cast<cudaStream_t>(stream));
        if (rp != ZZ_OK) return rp;
    }
    if (c->fp8 && nR > 0) {
        const int qr = quant_append(c, layer, static_cast<const __nv_bfloat16*>(d_k), static_cast<const __nv_bfloat16*>(d_v),
                                    h_n_new, nullptr, 1, static_cast<cudaStream_t>(stream));
        if (qr != ZZ_OK) return qr;
    }
    zz::AppendParams p;
    memset(&p, 0, sizeof p);
    p.skip_retrieval = (c->fp8 && nR > 0) ? 1 : 0;     // (the launch still moves the lengths)
    p.arena = c->d_arena();
    p.desc = c->d_desc(layer);
    p.len = c->d_len(layer);
    p.pos = c->d_pos(layer);
    p.counter = c->d_append_counter();
    p.k_new = static_cast<const __nv_bfloat16*>(d_k);
    p.v_new = static_cast<const __nv_bfloat16*>(d_v);
    p.head_list = c->d_heads(layer);
    p.page_table = c->paged ? c->d_table() : nullptr;
    p.nR = nR; p.Hkv = c->Hkv; p.ring = c->ring; p.S = c->S; p.W = c->W; p.B = c->B; p.D = c->D;
    int off = 0;
    for (int b = 0; b < c->B; ++b) {
        p.n_new[b] = h_n_new[b];
        p.tok_off[b] = off;
        off += h_n_new[b];
        const long long cand = h_n_new[b] < c->ring ? h_n_new[b] : c->ring;
        const long long work = ((long long)h_n_new[b] * nR + cand * nS) * (c->D >> 3);
        if (work > worst) worst = work;
    }
    const long long gx = (worst + 255) / 256;
    if (gx > 0x7fffffffLL) return ZZ_ERR_UNSUPPORTED;
    zz::prof_begin(zz::kProfAppend, static_cast<cudaStream_t>(stream));
    c->last_nowait = false;
    c->fresh_layer = layer;
    const cudaError_t ae = zz::launch_append(p, (int)gx, static_cast<cudaStream_t>(stream));
    zz::prof_end(zz::kProfAppend, static_cast<cudaStream_t>(stream));
    if (ae != cudaSuccess) return ZZ_ERR_CUDA;
    for (int b = 0; b < c->B; ++b) c->len[(size_t)layer * c->B + b] += h_n_new[b];
    return ZZ_OK;
}

int zz_decode_attn(zz_cache_t* c, int layer, const void* d_q, void* d_out, void* stream) {
    if (bad_layer(c, layer) || !d_q || !d_out) return ZZ_ERR_INVALID_ARG;
    if (((uintptr_t)d_q | (uintptr_t)d_out) & 15) return ZZ_ERR_INVALID_ARG;
    for (int b = 0; b < c->B; ++b)
        if (c->len[(size_t)layer * c->B + b] < 1) return ZZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(d_q);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(d_out);
    if (!c->mixed(layer)) {
        const int kind = c->nR[layer] ? ZZ_KIND_RETRIEVAL : ZZ_KIND_STREAMING;
        return launch_decode_group(c, layer, kind, q, out, 0, st, nullptr, nullptr, 0, c->decode_overlap ? 3 : 0);
    }
    // DuoAttention-style layer: gather the heads of each kind, one pass per kind, scatter back
    int r = regroup(c, layer, q, c->d_qc(), c->B, 1, st);
    const int ov = c->decode_overlap ? 3 : 0;
    if (r == ZZ_OK) r = launch_decode_group(c, layer, ZZ_KIND_RETRIEVAL, c->d_qc(), c->d_oc(), 0, st, nullptr, nullptr, 0, ov);
    if (r == ZZ_OK)
        r = launch_decode_group(c, layer, ZZ_KIND_STREAMING, c->d_qc(), c->d_oc(), c->nR[layer] * c->G, st, nullptr,
                                nullptr, 0, ov);
    if (r == ZZ_OK) r = regroup(c, layer, c->d_oc(), out, c->B, 0, st);
    return r;
}

static int decode_step_impl(zz_cache_t* c, int layer, const void* d_q, const void* d_k, const void* d_v,
                            void* d_out, void* stream, int overlap);

int zz_decode_step(zz_cache_t* c, int layer, const void* d_q, const void* d_k, const void* d_v, void* d_out,
                   void* stream) {
    return decode_step_impl(c, layer, d_q, d_k, d_v, d_out, stream, 0);
}

// overlap: the launch may start while the previous launch in the stream drains (exclusive layers
// only; the caller guarantees that launch belonged to another layer and did not produce q/k/v)
static int decode_step_impl(zz_cache_t* c, int layer, const void* d_q, const void* d_k, const void* d_v,
                            void* d_out, void* stream, int overlap) {
    if (bad_layer(c, layer) || !d_q || !d_k || !d_v || !d_out) return ZZ_ERR_INVALID_ARG;
    if (((uintptr_t)d_q | (uintptr_t)d_k | (uintptr_t)d_v | (uintptr_t)d_out) & 15) return ZZ_ERR_INVALID_ARG;
    const int nR = c->nR[layer];
    for (int b = 0; b < c->B; ++b) {
        const long long nl = (long long)c->len[(size_t)layer * c->B + b] + 1;
        if (nl > 0x7fffffffLL || (nR > 0 && nl > c->cap[b])) return ZZ_ERR_CAPACITY;
    }
    // the append is fused into the attention kernel: the new row is read from d_k/d_v, stored in
    // its slot and attended to by the same launch
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
        int32_t ones[ZZ_MAX_BATCH];
        for (int b = 0; b < c->B; ++b) ones[b] = 1;
        const int rp = reserve_pages(c, layer, layer + 1, ones, st);
        if (rp != ZZ_OK) return rp;
    }
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(d_q);
    const __nv_bfloat16* k = static_cast<const __nv_bfloat16*>(d_k);
    const __nv_bfloat16* v = static_cast<const __nv_bfloat16*>(d_v);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(d_out);
    int r;
    if (c->fp8 && nR > 0) {
        r = quant_append(c, layer, k, v, nullptr, nullptr, 1, st);
        if (r != ZZ_OK) return r;
        overlap = 0;       // the attention launch reads what the append wrote: plain stream order or a wait at entry
    }
    if (!c->mixed(layer)) {
        const int kind = nR ? ZZ_KIND_RETRIEVAL : ZZ_KIND_STREAMING;
        r = launch_decode_group(c, layer, kind, q, out, 0, st, k, v, 1,
                                overlap ? (c->decode_overlap > 2 ? 2 : c->decode_overlap) : (c->decode_overlap ? 3 : 0));
    } else {
        r = regroup(c, layer, q, c->d_qc(), c->B, 1, st);
        const int ov = c->decode_overlap ? 3 : 0;
        if (r == ZZ_OK) r = launch_decode_group(c, layer, ZZ_KIND_RETRIEVAL, c->d_qc(), c->d_oc(), 0, st, k, v, 0, ov);
        if (r == ZZ_OK)
            r = launch_decode_group(c, layer, ZZ_KIND_STREAMING, c->d_qc(), c->d_oc(), nR * c->G, st, k, v, 1, ov);
        if (r == ZZ_OK) r = regroup(c, layer, c->d_oc(), out, c->B, 0, st);
    }
    if (r != ZZ_OK) return r;
    for (int b = 0; b < c->B; ++b) c->len[(size_t)layer * c->B + b] += 1;
    return ZZ_OK;
}

int zz_decode_step_all(zz_cache_t* c, const void* d_q, const void* d_k, const void* d_v, void* d_out,
                       void* stream) {
    if (!c || !d_q || !d_k || !d_v || !d_out) return ZZ_ERR_INVALID_ARG;
    const size_t qs = (size_t)c->B * c->Hq * c->D * 2, ks = (size_t)c->B * c->Hkv * c->D * 2;
    // validate every layer before launching anything
    for (int l = 0; l < c->L; ++l)
        for (int b = 0; b < c->B; ++b)
            if (c->nR[l] > 0 && c->len[(size_t)l * c->B + b] + 1 > c->cap[b]) return ZZ_ERR_CAPACITY;
    {
        int32_t ones[ZZ_MAX_BATCH];
        for (int b = 0; b < c->B; ++b) ones[b] = 1;
        const int rp = reserve_pages(c, 0, c->L, ones, static_cast<cudaStream_t>(stream));
        if (rp != ZZ_OK) return rp;
    }
    // Equal lengths in every layer: one launch per kind of work instead of one (or four) per layer
    // (blockIdx.y = layer).  The layers are independent (own stores, lengths, scratch and output
    // slice; q/k/v of all layers are inputs of the call), so a launch over many layers only removes
    // launch boundaries: no ramp-up and tail per layer, and the ~3 us per launch that a streaming
    // layer's few CTAs cannot fill.  Mixed layers join when they all have the same number of
    // retrieval heads (one split plan serves them all): one regrouping launch before and one after,
    // and their two passes ride in grids of their own.
    bool same_len = c->decode_overlap == 3 && (c->n_mixed == 0 || c->mixed_same_nR);
    for (int l = 1; l < c->L && same_len; ++l)
        for (int b = 0; b < c->B; ++b)
            if (c->len[(size_t)l * c->B + b] != c->len[b]) same_len = false;
    if (same_len) {
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        if (((uintptr_t)d_q | (uintptr_t)d_k | (uintptr_t)d_v | (uintptr_t)d_out) & 15) return ZZ_ERR_INVALID_ARG;
        const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(d_q);
        const __nv_bfloat16* k = static_cast<const __nv_bfloat16*>(d_k);
        const __nv_bfloat16* v = static_cast<const __nv_bfloat16*>(d_v);
        __nv_bfloat16* out = static_cast<__nv_bfloat16*>(d_out);
        // Order: [regroup q of the mixed layers], the short streaming grids, then the retrieval
        // grids, [regroup the mixed layers' outputs].  The first decode grid is an ordinary launch
        // (it starts after the regrouping copy has completed).  Every later grid is a programmatic
        // launch: it starts while its predecessor's CTAs run and executes griddepcontrol.wait after
        // its main loop, before it touches the split scratch, the output or the lengths.  A grid
        // therefore completes only after its predecessor has, so the chain completes in order, the
        // two passes of a mixed layer never share scratch at the same time, and whatever follows in
        // the stream only has to wait for the last launch.
        const int* ids = c->d_layer_ids();
        const int oS = c->n_excl_R, oM = c->n_excl_R + c->n_excl_S;
        int r = ZZ_OK;
        bool first = true;
        if (c->fp8) {
            // the step's rows of every retrieval head, quantised into their slots before anything attends
            if (c->n_excl_R > 0) r = quant_append(c, c->layer_ids[0], k, v, nullptr, ids, c->n_excl_R, st);
            if (r == ZZ_OK && c->n_mixed > 0) r = quant_append(c, c->layer_ids[oM], k, v, nullptr, ids + oM, c->n_mixed, st);
        }
        if (r == ZZ_OK && c->n_mixed > 0) r = regroup(c, -1, q, c->d_dqc(), (long long)c->n_mixed * c->B, 1, st);
        if (r == ZZ_OK && c->n_excl_S > 0) {
            r = launch_decode_group(c, c->layer_ids[oS], ZZ_KIND_STREAMING, q, out, 0, st, k, v, 1, first ? 0 : 1,
                                    ids + oS, c->n_excl_S);
            first = false;
        }
        if (r == ZZ_OK && c->n_mixed > 0) {
            const int lm = c->layer_ids[oM];
            r = launch_decode_group(c, lm, ZZ_KIND_STREAMING, c->d_dqc(), c->d_doc(), c->nR[lm] * c->G, st, k, v, 0,
                                    first ? 0 : 1, ids + oM, c->n_mixed);
            first = false;
            // the retrieval pass is the layer's last: it publishes the new lengths
            if (r == ZZ_OK)
                r = launch_decode_group(c, lm, ZZ_KIND_RETRIEVAL, c->d_dqc(), c->d_doc(), 0, st, k, v, 1, 1, ids + oM,
                                        c->n_mixed);
        }
        if (r == ZZ_OK && c->n_excl_R > 0)
            r = launch_decode_group(c, c->layer_ids[0], ZZ_KIND_RETRIEVAL, q, out, 0, st, k, v, 1, first ? 0 : 1, ids,
                                    c->n_excl_R);
        if (r == ZZ_OK && c->n_mixed > 0) r = regroup(c, -1, c->d_doc(), out, (long long)c->n_mixed * c->B, 0, st);
        if (r != ZZ_OK) return r;
        for (size_t i = 0; i < c->len.size(); ++i) c->len[i] += 1;
        return ZZ_OK;
    }
    for (int l = 0; l < c->L; ++l) {
        // q/k/v of every layer are inputs of this call, and layer l's launch reads nothing that layer
        // l-1's launches write before its griddepcontrol.wait, so consecutive layers may overlap
        const int r = decode_step_impl(c, l, static_cast<const char*>(d_q) + l * qs,
                                       static_cast<const char*>(d_k) + l * ks,
                                       static_cast<const char*>(d_v) + l * ks,
                                       static_cast<char*>(d_out) + l * qs, stream, l > 0);
        if (r != ZZ_OK) return r;
    }
    return ZZ_OK;
}

int zz_profile_enable(int period) {
    if (period < 0) return ZZ_ERR_INVALID_ARG;
    zz::g_prof.period = period;
    for (int i = 0; i < zz::kProfKinds; ++i) zz::g_prof.seen[i] = 0;
    return ZZ_OK;
}

int zz_profile_read(int kind, int64_t* launches, double* total_ms, int reset) {
    if (kind < 0 || kind >= zz::kProfKinds || !launches || !total_ms) return ZZ_ERR_INVALID_ARG;
    long long n = 0;
    double ms = 0.0;
    for (const auto& r : zz::g_prof.recs) {
        if (r.kind != kind) continue;
        if (cudaEventSynchronize(r.e1) != cudaSuccess) return ZZ_ERR_CUDA;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, r.e0, r.e1) != cudaSuccess) return ZZ_ERR_CUDA;
        ms += t;
        ++n;
    }
    *launches = n;
    *total_ms = ms;
    if (reset) {
        for (const auto& r : zz::g_prof.recs) {
            zz::g_prof.pool.push_back(r.e0);
            zz::g_prof.pool.push_back(r.e1);
        }
        zz::g_prof.recs.clear();
    }
    return ZZ_OK;
}

int zz_prefill_attn(zz_cache_t* c, int layer, const void* d_q, const void* d_k, const void* d_v, void* d_out,
                    const int32_t* h_n_new, void* stream) {
    if (bad_layer(c, layer) || !d_q || !d_k || !d_v || !d_out || !h_n_new) return ZZ_ERR_INVALID_ARG;
    if (((uintptr_t)d_q | (uintptr_t)d_k | (uintptr_t)d_v | (uintptr_t)d_out) & 15) return ZZ_ERR_INVALID_ARG;
    long long total = 0;
    for (int b = 0; b < c->B; ++b) {
        if (h_n_new[b] < 0) return ZZ_ERR_INVALID_ARG;
        if ((long long)c->len[(size_t)layer * c->B + b] + h_n_new[b] > 0x7fffffffLL) return ZZ_ERR_CAPACITY;
        total += h_n_new[b];
    }
    if (total == 0) return ZZ_OK;
    if (!c->have_tmap_arena) return ZZ_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(d_q);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(d_out);
    alignas(64) CUtensorMap tq, tk, tv;
    if (!encode_rows3d(&tk, d_k, total, c->Hkv, c->D) || !encode_rows3d(&tv, d_v, total, c->Hkv, c->D)) return ZZ_ERR_CUDA;
    if (!c->mixed(layer)) {
        if (!encode_rows3d(&tq, q, total, c->Hq, c->D)) return ZZ_ERR_CUDA;
        const int kind = c->nR[layer] ? ZZ_KIND_RETRIEVAL : ZZ_KIND_STREAMING;
        return launch_prefill_group(c, layer, kind, &tq, &tk, &tv, out, 0, h_n_new, st);
    }
    if (total > c->max_new) return ZZ_ERR_WORKSPACE;
    if (!encode_rows3d(&tq, c->d_qc(), total, c->Hq, c->D)) return ZZ_ERR_CUDA;
    int r = regroup(c, layer, q, c->d_qc(), total, 1, st);
    if (r == ZZ_OK) r = launch_prefill_group(c, layer, ZZ_KIND_RETRIEVAL, &tq, &tk, &tv, c->d_oc(), 0, h_n_new, st);
    if (r == ZZ_OK)
        r = launch_prefill_group(c, layer, ZZ_KIND_STREAMING, &tq, &tk, &tv, c->d_oc(), c->nR[layer] * c->G,
                                 h_n_new, st);
    if (r == ZZ_OK) r = regroup(c, layer, c->d_oc(), out, total, 0, st);
    return r;
}

size_t zz_stage_bytes(const zz_cache_t* c, int64_t n_tokens) {
    if (!c || n_tokens < 0) return 0;
    const size_t qb = align_up((size_t)n_tokens * c->Hq * c->D * 2);
    const size_t kb = align_up((size_t)n_tokens * c->Hkv * c->D * 2);
    return 2 * qb + 2 * kb;
}

static int run_host(zz_cache_t* c, int layer, const void* h_q, const void* h_k, const void* h_v, void* h_out,
                    const int32_t* n_new, void* d_stage, size_t stage_bytes, void* stream, bool decode) {
    if (bad_layer(c, layer) || !h_q || !h_k || !h_v || !h_out || !d_stage || !n_new) return ZZ_ERR_INVALID_ARG;
    long long total = 0;
    for (int b = 0; b < c->B; ++b) {
        if (n_new[b] < 0) return ZZ_ERR_INVALID_ARG;
        total += n_new[b];
    }
    if (stage_bytes < zz_stage_bytes(c, total)) return ZZ_ERR_WORKSPACE;
    if ((uintptr_t)d_stage % kAlign) return ZZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t qbytes = (size_t)total * c->Hq * c->D * 2, kbytes = (size_t)total * c->Hkv * c->D * 2;
    const size_t qb = align_up(qbytes), kb = align_up(kbytes);
    unsigned char* s = static_cast<unsigned char*>(d_stage);
    void* dq = s; void* dk = s + qb; void* dv = s + qb + kb; void* dout = s + qb + 2 * kb;
    if (total == 0) return ZZ_OK;
    if (cudaMemcpyAsync(dq, h_q, qbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (cudaMemcpyAsync(dk, h_k, kbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (cudaMemcpyAsync(dv, h_v, kbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZZ_ERR_CUDA;
    int r;
    if (decode) {
        r = zz_decode_step(c, layer, dq, dk, dv, dout, stream);
    } else {
        r = zz_prefill_attn(c, layer, dq, dk, dv, dout, n_new, stream);
        if (r == ZZ_OK) r = zz_kv_append(c, layer, dk, dv, n_new, stream);
    }
    if (r != ZZ_OK) return r;
    if (cudaMemcpyAsync(h_out, dout, qbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZZ_ERR_CUDA;
    return ZZ_OK;
}

int zz_decode_step_host(zz_cache_t* c, int layer, const void* h_q, const void* h_k, const void* h_v,
                        void* h_out, void* d_stage, size_t stage_bytes, void* stream) {
    if (!c) return ZZ_ERR_INVALID_ARG;
    int32_t ones[ZZ_MAX_BATCH];
    for (int b = 0; b < c->B; ++b) ones[b] = 1;
    return run_host(c, layer, h_q, h_k, h_v, h_out, ones, d_stage, stage_bytes, stream, true);
}

int zz_decode_step_all_host(zz_cache_t* c, const void* h_q, const void* h_k, const void* h_v, void* h_out,
                            void* d_stage, size_t stage_bytes, void* stream) {
    if (!c || !h_q || !h_k || !h_v || !h_out || !d_stage) return ZZ_ERR_INVALID_ARG;
    const long long total = (long long)c->L * c->B;
    if (stage_bytes < zz_stage_bytes(c, total)) return ZZ_ERR_WORKSPACE;
    if ((uintptr_t)d_stage % kAlign) return ZZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t qbytes = (size_t)total * c->Hq * c->D * 2, kbytes = (size_t)total * c->Hkv * c->D * 2;
    const size_t qb = align_up(qbytes), kb = align_up(kbytes);
    unsigned char* s = static_cast<unsigned char*>(d_stage);
    void* dq = s; void* dk = s + qb; void* dv = s + qb + kb; void* dout = s + qb + 2 * kb;
    const char* hq = static_cast<const char*>(h_q);
    if (static_cast<const char*>(h_k) == hq + qbytes && static_cast<const char*>(h_v) == hq + qbytes + kbytes &&
        qb == qbytes && kb == kbytes) {
        // q, k and v lie back to back on the host (and so they do in the staging buffer): one copy
        if (cudaMemcpyAsync(dq, h_q, qbytes + 2 * kbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZZ_ERR_CUDA;
    } else {
        if (cudaMemcpyAsync(dq, h_q, qbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZZ_ERR_CUDA;
        if (cudaMemcpyAsync(dk, h_k, kbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZZ_ERR_CUDA;
        if (cudaMemcpyAsync(dv, h_v, kbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZZ_ERR_CUDA;
    }
    const int r = zz_decode_step_all(c, dq, dk, dv, dout, stream);
    if (r != ZZ_OK) return r;
    if (cudaMemcpyAsync(h_out, dout, qbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZZ_ERR_CUDA;
    return ZZ_OK;
}

int zz_prefill_host(zz_cache_t* c, int layer, const void* h_q, const void* h_k, const void* h_v, void* h_out,
                    const int32_t* h_n_new, void* d_stage, size_t stage_bytes, void* stream) {
    return run_host(c, layer, h_q, h_k, h_v, h_out, h_n_new, d_stage, stage_bytes, stream, false);
}

int zz_cache_export_shape(const zz_cache_t* c, int layer, int seq, int kind, int32_t* n_heads,
                          int32_t* n_slots) {
    if (bad_layer(c, layer) || seq < 0 || seq >= c->B || (kind != 0 && kind != 1) || !n_heads || !n_slots)
        return ZZ_ERR_INVALID_ARG;
    *n_heads = (kind == ZZ_KIND_RETRIEVAL) ? c->nR[layer] : c->Hkv - c->nR[layer];
    *n_slots = (kind == ZZ_KIND_RETRIEVAL) ? c->cap[seq] : c->ring;
    return ZZ_OK;
}

int zz_cache_export(zz_cache_t* c, int layer, int seq, int kind, void* h_k, void* h_v, int32_t* h_pos,
                    int32_t* h_len, void* stream) {
    int32_t nh, ns;
    const int r = zz_cache_export_shape(c, layer, seq, kind, &nh, &ns);
    if (r != ZZ_OK) return r;
    if (!h_k || !h_v || !h_pos || !h_len) return ZZ_ERR_INVALID_ARG;
    if (c->fp8 && kind == ZZ_KIND_RETRIEVAL) return ZZ_ERR_UNSUPPORTED;   // use zz_cache_export_fp8
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const SeqDesc& d = c->desc[(size_t)layer * c->B + seq];
    const size_t bytes = (size_t)nh * ns * c->D * 2;
    cudaError_t e = cudaSuccess;
    if (bytes && c->paged && kind == ZZ_KIND_RETRIEVAL) {
        // page by page into the contiguous [head][slot][128] host layout; slots without a page are left alone
        const size_t lb = (size_t)layer * c->B + seq;
        for (int g = 0; g < c->pages_of[lb] && e == cudaSuccess; ++g)
            for (int h = 0; h < nh && e == cudaSuccess; ++h) {
                const long long page = c->h_table[d.tbl + g * nh + h];
                const int rows = (ns - g * zz::kPageTokens < zz::kPageTokens) ? ns - g * zz::kPageTokens : zz::kPageTokens;
                const size_t ho = ((size_t)h * ns + (size_t)g * zz::kPageTokens) * kD * 2;
                e = cudaMemcpyAsync(static_cast<char*>(h_k) + ho, c->d_arena() + d.k_off[kind] + page * zz::kPageElems,
                                    (size_t)rows * kD * 2, cudaMemcpyDeviceToHost, st);
                if (e == cudaSuccess)
                    e = cudaMemcpyAsync(static_cast<char*>(h_v) + ho,
                                        c->d_arena() + d.v_off[kind] + page * zz::kPageElems, (size_t)rows * kD * 2,
                                        cudaMemcpyDeviceToHost, st);
            }
    } else if (bytes) {
        e = cudaMemcpyAsync(h_k, c->d_arena() + d.k_off[kind], bytes, cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(h_v, c->d_arena() + d.v_off[kind], bytes, cudaMemcpyDeviceToHost, st);
    }
    int dev_len = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&dev_len, c->d_len(layer) + seq, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && kind == ZZ_KIND_STREAMING)
        e = cudaMemcpyAsync(h_pos, c->d_pos(layer) + (size_t)seq * c->ring, (size_t)c->ring * sizeof(int),
                            cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return ZZ_ERR_CUDA;
    *h_len = dev_len;
    if (kind == ZZ_KIND_RETRIEVAL)
        for (int i = 0; i < ns; ++i) h_pos[i] = (i < dev_len) ? i : -1;
    return ZZ_OK;
}

int zz_cache_import(zz_cache_t* c, int layer, int seq, int kind, const void* h_k, const void* h_v,
                    const int32_t* h_pos, int32_t len, void* stream) {
    int32_t nh, ns;
    const int r = zz_cache_export_shape(c, layer, seq, kind, &nh, &ns);
    if (r != ZZ_OK) return r;
    if (!h_k || !h_v || !h_pos || len < 0) return ZZ_ERR_INVALID_ARG;
    if (c->fp8 && kind == ZZ_KIND_RETRIEVAL) return ZZ_ERR_UNSUPPORTED;   // use zz_cache_import_fp8
    if (kind == ZZ_KIND_RETRIEVAL && len > ns) return ZZ_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const SeqDesc& d = c->desc[(size_t)layer * c->B + seq];
    const size_t bytes = (size_t)nh * ns * c->D * 2;
    cudaError_t e = cudaSuccess;
    if (bytes && c->paged && kind == ZZ_KIND_RETRIEVAL) {
        const size_t lb = (size_t)layer * c->B + seq;
        int32_t add[ZZ_MAX_BATCH] = {0};
        add[seq] = len > c->len[lb] ? len - c->len[lb] : 0;
        const int rp = reserve_pages(c, layer, layer + 1, add, st);
        if (rp != ZZ_OK) return rp;
        const int blocks = (len + zz::kPageTokens - 1) / zz::kPageTokens;
        for (int g = 0; g < blocks && e == cudaSuccess; ++g)
            for (int h = 0; h < nh && e == cudaSuccess; ++h) {
                const long long page = c->h_table[d.tbl + g * nh + h];
                const int rows = (ns - g * zz::kPageTokens < zz::kPageTokens) ? ns - g * zz::kPageTokens : zz::kPageTokens;
                const size_t ho = ((size_t)h * ns + (size_t)g * zz::kPageTokens) * kD * 2;
                e = cudaMemcpyAsync(c->d_arena() + d.k_off[kind] + page * zz::kPageElems,
                                    static_cast<const char*>(h_k) + ho, (size_t)rows * kD * 2, cudaMemcpyHostToDevice, st);
                if (e == cudaSuccess)
                    e = cudaMemcpyAsync(c->d_arena() + d.v_off[kind] + page * zz::kPageElems,
                                        static_cast<const char*>(h_v) + ho, (size_t)rows * kD * 2,
                                        cudaMemcpyHostToDevice, st);
            }
    } else if (bytes) {
        e = cudaMemcpyAsync(c->d_arena() + d.k_off[kind], h_k, bytes, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaMemcpyAsync(c->d_arena() + d.v_off[kind], h_v, bytes, cudaMemcpyHostToDevice, st);
    }
    if (e == cudaSuccess && kind == ZZ_KIND_STREAMING)
        e = cudaMemcpyAsync(c->d_pos(layer) + (size_t)seq * c->ring, h_pos, (size_t)c->ring * sizeof(int),
                            cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(c->d_len(layer) + seq, &len, sizeof(int), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return ZZ_ERR_CUDA;
    c->len[(size_t)layer * c->B + seq] = len;
    return ZZ_OK;
}

// FP8 retrieval group of (layer, seq): codes [heads][cap][128] and scale bytes [heads][cap], both ways
static int fp8_copy(zz_cache_t* c, int layer, int seq, void* h_k, void* h_v, void* h_ks, void* h_vs, bool to_host,
                    cudaStream_t st) {
    const SeqDesc& d = c->desc[(size_t)layer * c->B + seq];
    const int nh = c->nR[layer], cap = d.cap, cap16 = zz::fp8_cap16(cap);
    unsigned char* kc = c->arena + 2 * d.k_off[ZZ_KIND_RETRIEVAL];
    unsigned char* vc = c->arena + 2 * d.v_off[ZZ_KIND_RETRIEVAL];
    unsigned char* ks = c->arena + zz::fp8_kscale_byte_off(d.v_off[ZZ_KIND_RETRIEVAL], nh, cap);
    unsigned char* vs = ks + (size_t)nh * cap16;
    const size_t cb = (size_t)nh * cap * kD;
    const cudaMemcpyKind kd = to_host ? cudaMemcpyDeviceToHost : cudaMemcpyHostToDevice;
    cudaError_t e = cudaSuccess;
    if (cb) {
        e = to_host ? cudaMemcpyAsync(h_k, kc, cb, kd, st) : cudaMemcpyAsync(kc, h_k, cb, kd, st);
        if (e == cudaSuccess) e = to_host ? cudaMemcpyAsync(h_v, vc, cb, kd, st) : cudaMemcpyAsync(vc, h_v, cb, kd, st);
        // scale rows are padded to a multiple of 16 on the device, packed [heads][cap] on the host
        if (e == cudaSuccess)
            e = to_host ? cudaMemcpy2DAsync(h_ks, cap, ks, cap16, cap, nh, kd, st) : cudaMemcpy2DAsync(ks, cap16, h_ks, cap, cap, nh, kd, st);
        if (e == cudaSuccess)
            e = to_host ? cudaMemcpy2DAsync(h_vs, cap, vs, cap16, cap, nh, kd, st) : cudaMemcpy2DAsync(vs, cap16, h_vs, cap, cap, nh, kd, st);
    }
    return e == cudaSuccess ? ZZ_OK : ZZ_ERR_CUDA;
}

int zz_cache_export_fp8(zz_cache_t* c, int layer, int seq, void* h_k_codes, void* h_v_codes, void* h_k_scale,
                        void* h_v_scale, int32_t* h_len, void* stream) {
    if (bad_layer(c, layer) || seq < 0 || seq >= c->B || !h_k_codes || !h_v_codes || !h_k_scale || !h_v_scale || !h_len)
        return ZZ_ERR_INVALID_ARG;
    if (!c->fp8) return ZZ_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int r = fp8_copy(c, layer, seq, h_k_codes, h_v_codes, h_k_scale, h_v_scale, true, st);
    if (r != ZZ_OK) return r;
    int dev_len = 0;
    if (cudaMemcpyAsync(&dev_len, c->d_len(layer) + seq, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZZ_ERR_CUDA;
    *h_len = dev_len;
    return ZZ_OK;
}

int zz_cache_import_fp8(zz_cache_t* c, int layer, int seq, const void* h_k_codes, const void* h_v_codes,
                        const void* h_k_scale, const void* h_v_scale, int32_t len, void* stream) {
    if (bad_layer(c, layer) || seq < 0 || seq >= c->B || !h_k_codes || !h_v_codes || !h_k_scale || !h_v_scale || len < 0)
        return ZZ_ERR_INVALID_ARG;
    if (!c->fp8) return ZZ_ERR_UNSUPPORTED;
    if (c->nR[layer] > 0 && len > c->cap[seq]) return ZZ_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int r = fp8_copy(c, layer, seq, const_cast<void*>(h_k_codes), const_cast<void*>(h_v_codes), const_cast<void*>(h_k_scale),
                     const_cast<void*>(h_v_scale), false, st);
    if (r != ZZ_OK) return r;
    if (cudaMemcpyAsync(c->d_len(layer) + seq, &len, sizeof(int), cudaMemcpyHostToDevice, st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZZ_ERR_CUDA;
    c->len[(size_t)layer * c->B + seq] = len;
    return ZZ_OK;
}

int zz_selftest_wait_timeout(zz_cache_t* c, int32_t max_polls, void* stream) {
    if (!c || max_polls < 1 || max_polls > (1 << 16)) return ZZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the flag sits in the spare bytes of the status section (word 0 status, word 16 append counter)
    int* gave_up = c->d_status() + 32;
    if (cudaMemsetAsync(gave_up, 0, sizeof(int), st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (zz::launch_wait_probe(c->d_status(), (unsigned int)max_polls, gave_up, st) != cudaSuccess) return ZZ_ERR_CUDA;
    int v = 0;
    if (cudaMemcpyAsync(&v, gave_up, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZZ_ERR_CUDA;
    return v == 1 ? ZZ_OK : ZZ_ERR_CUDA;
}

int zz_get_last_status(zz_cache_t* c, void* stream) {
    if (!c) return ZZ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int v = 0;
    if (cudaMemcpyAsync(&v, c->d_status(), sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (v != 0) {
        if (cudaMemsetAsync(c->d_status(), 0, sizeof(int), st) != cudaSuccess) return ZZ_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return ZZ_ERR_CUDA;
    }
    return v;
}

}  // extern "C"
