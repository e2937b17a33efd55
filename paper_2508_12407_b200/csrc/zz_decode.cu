// Decode attention: one query token per sequence over a KV store.
//
// The same kernel serves retrieval layers (split-sequence flash decoding over the whole
// append-only store) and streaming layers (a single pass over the occupied ring slots in
// physical order: after an append the ring holds exactly the visible set, and the occupied
// slots are always the first min(len, S+W) ones).
//
// Work item = (sequence, KV head of the group, token range).  The G query heads that share a
// KV head are the rows of one 16-row MMA tile, so every K/V byte is read from HBM once and
// used by all of them.  Each warp streams its own 16-token blocks through a private
// multi-stage cp.async pipeline (16-byte coalesced loads, zero-filled past the range end),
// keeps a private online-softmax state, and the warps, then the splits, are merged with the
// usual (max, sum, weighted output) rule.  The last CTA of a (sequence, head) to finish does
// the split merge, so there is no second launch.
//
// The roofline of this kernel is HBM bandwidth: 2 * 128 * 2 bytes per token and KV head.
//
// Also here: the append of the step's new token fused into the launch (its row is taken from the
// caller's tensors, stored in its slot and attended to; the kernel refuses by itself when a
// retrieval store has no room, for launches replayed from a CUDA graph), a grid over several
// layers (blockIdx.y), paged retrieval stores (separate instantiations), L2 policy hints on the
// K/V loads, and the programmatic-dependent-launch hooks that let consecutive launches overlap.
#include <cstring>

#include "zz_decode_merge.cuh"

namespace zz {

namespace {

constexpr int kBlk = 16;                       // tokens per warp step
constexpr int kWarpSmem = 24 * 1024;           // per warp: 3 stages of 2 x 4 KiB at head_dim 128, 6 stages of 2 x 2 KiB at 64
// 4 warps: 96 KiB, two CTAs per SM (long contexts); 8 warps: 192 KiB, one CTA per SM (short
// stores, where the per-warp chain of dependent steps is what costs)

// Issue the loads of one 16-token block (K and V rows of one head) into a stage.
// Row r, 16-byte piece c lands at r*256 + ((c ^ (r & 7)) * 16): conflict-free for ldmatrix.
// Slot `new_slot` (if inside the block) is the token being appended by this very launch: its
// row comes from the caller's k_new/v_new instead of the store.
template <int HD>
__device__ __forceinline__ void load_block(uint32_t stage_k, uint32_t stage_v, const __nv_bfloat16* kbase,
                                           const __nv_bfloat16* vbase, int tok0, int tok_end, int lane,
                                           int new_slot, const __nv_bfloat16* knew, const __nv_bfloat16* vnew,
                                           uint64_t policy) {
    constexpr int kRowB = HD * 2;              // bytes of a row (HD / 8 sixteen-byte pieces)
    if (HD == 64) {
        // 128-byte rows: lane -> (row it * 4 + lane / 8, piece lane % 8), pieces XOR-swizzled by row
        const bool whole = tok0 + kBlk <= tok_end && (new_slot < tok0 || new_slot >= tok0 + kBlk);
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int r = it * 4 + (lane >> 3), c = lane & 7;
            const int tok = tok0 + r;
            const int ok = tok < tok_end;
            const long long off = (long long)(ok ? tok : tok0) * HD + c * 8;
            const uint32_t so = r * kRowB + ((c ^ (r & 7)) << 4);
            if (whole) {
                cp_async16_full(stage_k + so, kbase + off, policy);
                cp_async16_full(stage_v + so, vbase + off, policy);
            } else {
                const bool fresh = tok == new_slot;
                cp_async16(stage_k + so, fresh ? knew + c * 8 : kbase + off, ok ? 16 : 0);
                cp_async16(stage_v + so, fresh ? vnew + c * 8 : vbase + off, ok ? 16 : 0);
            }
        }
        return;
    }
    if (tok0 + kBlk <= tok_end && (new_slot < tok0 || new_slot >= tok0 + kBlk)) {
        // Whole block from the store (all but the edge blocks of a range): one pointer per lane, every
        // further address a constant away.  Row r = 2*it + r0 swizzles with (r & 7) = 2*(it & 3) + r0,
        // which touches bits the two terms do not share, so it folds into one XOR per iteration.
        const int r0 = lane >> 4, c = lane & 15;
        const long long off0 = (long long)(tok0 + r0) * HD + c * 8;
        const __nv_bfloat16* kp = kbase + off0;
        const __nv_bfloat16* vp = vbase + off0;
        const uint32_t so0 = r0 * kRowB + ((c ^ r0) << 4);
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const uint32_t so = (so0 ^ ((it & 3) << 5)) + it * 2 * kRowB;
            cp_async16_full(stage_k + so, kp + it * 2 * HD, policy);
            cp_async16_full(stage_v + so, vp + it * 2 * HD, policy);
        }
        return;
    }
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        const int idx = it * 32 + lane;
        const int r = idx >> 4, c = idx & 15;
        const int tok = tok0 + r;
        const int ok = tok < tok_end;
        const long long off = (long long)(ok ? tok : tok0) * HD + c * 8;
        const uint32_t so = r * kRowB + ((c ^ (r & 7)) << 4);
        const bool fresh = tok == new_slot;
        cp_async16(stage_k + so, fresh ? knew + c * 8 : kbase + off, ok ? 16 : 0);
        cp_async16(stage_v + so, fresh ? vnew + c * 8 : vbase + off, ok ? 16 : 0);
    }
}

// HI = group size above 8 (rows 8..15 of the tile carry query heads too).
// kPaged: the retrieval store is paged (compiled apart, so that the contiguous kernel carries none of it).
// HD = head_dim (128, or 64: half the row bytes, twice the stages, half the MMA steps and accumulators).
template <bool HI, int kWarps, bool kPaged, int HD>
__global__ void __launch_bounds__(kWarps * 32, 8 / kWarps) decode_kernel(const DecodeParams p) {
    constexpr int kRowB = HD * 2;                          // bytes of a K or V row
    constexpr int kStageBytes = kBlk * kRowB;              // K (and as much of V) per stage
    constexpr int kStages = kWarpSmem / (2 * kStageBytes); // 3 at head_dim 128, 6 at 64: the same bytes in flight
    constexpr int kKSteps = HD / 16;                       // 16-dim MMA steps of Q K^T, 16-column pairs of P V
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ int s_is_last;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = lane >> 2, tig = lane & 3;

    // (a launch that waits at entry lets its dependents go after that wait, further down)
    if (p.gdc_wait != 2) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- which layer (a launch may cover several layers of a decode step: blockIdx.y) -----------
    const int li = p.layer_ids ? p.layer_ids[blockIdx.y] : 0;
    int* const len_p = p.len + (long long)li * p.st_len;
    int* const pos_p = p.pos + (long long)li * p.st_pos;
    const __nv_bfloat16* const q_p = p.q + (long long)li * p.st_q;
    __nv_bfloat16* const out_p = p.out + (long long)li * p.st_q;
    const __nv_bfloat16* const k_new_p = p.k_new ? p.k_new + (long long)li * p.st_kv : nullptr;
    const __nv_bfloat16* const v_new_p = p.v_new ? p.v_new + (long long)li * p.st_kv : nullptr;
    const int* const head_list_p = p.head_list + (long long)li * p.n_kv_total;
    unsigned int* const counters_p = p.counters + (long long)li * p.st_cnt;
    unsigned int* const seq_counters_p = p.seq_counters + (long long)li * p.st_cnt;
    float* const part_o_p = p.part_o + (long long)li * p.st_part * HD;
    float* const part_ml_p = p.part_ml + (long long)li * p.st_part * 2;

    // ---- which work item (launch parameters only) ----------------------------------------
    const int item = blockIdx.x;
    int b = 0;
    while (b + 1 < p.B && item >= p.split_start[b + 1] * p.Hg) ++b;
    const int local = item - p.split_start[b] * p.Hg;
    const int hg = local % p.Hg;
    const int split = local / p.Hg;
    const int nsplit = p.split_start[b + 1] - p.split_start[b];

    // A plan with more splits than the merge rows hold is refused, not run: every CTA of the launch
    // sees the same plan and returns before it touches a store, the scratch or the output.
    if (nsplit > p.max_splits || p.max_splits > kDecodeMaxSplits) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, ZZ_ERR_UNSUPPORTED);
        return;
    }

    // (read beside the store addresses unless the launch has to wait first)
    const int len_nowait = (p.gdc_wait != 2) ? len_p[b] : 0;
    // store addresses: written when the cache was created, never by a launch
    const SeqDesc sd = p.layer_ids ? p.desc_table[(long long)li * p.B + b] : p.sd[b];
    const long long slots_per_head = (p.kind == ZZ_KIND_RETRIEVAL) ? sd.cap : p.ring;
    // paged retrieval store: the bases are the pool's; each 16-token block adds its page's offset
    constexpr bool paged = kPaged;
    __nv_bfloat16* kbase = p.arena + sd.k_off[p.kind] + (paged ? 0ll : (long long)hg * slots_per_head * HD);
    __nv_bfloat16* vbase = p.arena + sd.v_off[p.kind] + (paged ? 0ll : (long long)hg * slots_per_head * HD);
    const uint32_t wbase = smem_u32(smem) + warp * kWarpSmem;
    // L2 policy of the K/V loads: a retrieval store is streamed once per step and should not push
    // anything out of the L2 (evict first); the rings of the streaming layers are read again by the
    // next step and together fit the L2 (evict last)
    uint64_t l2_policy;
    if (p.kind == ZZ_KIND_RETRIEVAL)
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(l2_policy));
    else
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(l2_policy));

    // Programmatic dependent launch (no-ops in an ordinary launch): the next launch in the stream
    // may start as soon as every CTA of this one is running, and fills the SMs this launch leaves
    // idle in its tail.  A launch that shares anything with its predecessor (gdc_wait) touches it
    // only after griddepcontrol.wait below; the layers of one decode step share nothing (own
    // stores, lengths, split workspace and output slice) and run without that wait.
    //
    // A launch that waits at entry (gdc_wait == 2) still has something it may do first.  A retrieval
    // store is append-only, so the rows that were complete before the previous launch began
    // (early_len, from the host) cannot change under it: the first stages of the K/V pipeline are
    // fetched before the wait, while the previous launch drains, whenever their blocks lie wholly
    // below that length.  The plan (chunk, split_start) is in the launch parameters, so the blocks
    // are known without the device length; the length, q and the step's token are read after the wait.
    unsigned pre = 0;           // bit s: stage s of the prologue is already in flight
    if (p.gdc_wait == 2) {
        if constexpr (!kPaged) {
            if (p.kind == ZZ_KIND_RETRIEVAL) {
                const int ne = p.early_len[b];
                const int e0 = split * p.chunk[b];
                const int e1 = (split == nsplit - 1) ? ne : min(ne, e0 + p.chunk[b]);
#pragma unroll
                for (int s = 0; s < kStages - 1; ++s) {
                    const int tok0 = e0 + (warp + s * kWarps) * kBlk;
                    if (tok0 + kBlk <= e1) {
                        load_block<HD>(wbase + s * 2 * kStageBytes, wbase + s * 2 * kStageBytes + kStageBytes, kbase,
                                       vbase, tok0, e1, lane, -1, nullptr, nullptr, l2_policy);
                        pre |= 1u << s;
                    }
                    cp_async_commit();
                }
            }
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");   // before anything a launch may have written is read
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }

    const bool fused = k_new_p != nullptr;
    const int len_old = (p.gdc_wait != 2) ? len_nowait : len_p[b];
    if (pre != 0 && len_old < p.early_len[b]) {
        // the store is shorter than the host believed (lengths reset under a replayed launch): what was
        // fetched early may lie past its end; let those copies land and fill the stages again below
        cp_async_wait<0>();
        __syncwarp();
        pre = 0;
    }
    const int len = len_old + (fused ? 1 : 0);
    const int n = (p.kind == ZZ_KIND_RETRIEVAL) ? len : min(len, p.ring);
    const int* const tbl = paged ? p.page_table + sd.tbl + hg : nullptr;   // entry of page g: tbl[g * Hg]
    int new_slot = -1;
    const __nv_bfloat16* knew = nullptr;
    const __nv_bfloat16* vnew = nullptr;
    if (fused && p.kind == ZZ_KIND_RETRIEVAL) {
        // Room for the appended row?  The host checks this before it launches; a launch replayed
        // from a CUDA graph has no host check, so the kernel refuses by itself: every CTA of the
        // sequence sees the same length and returns before it touches the store, the scratch or the
        // output, and the status word tells the host.
        bool room = len_old < sd.cap;
        if (paged && room) room = tbl[(len_old >> 7) * p.Hg] >= 0;
        if (!room) {
            if (threadIdx.x == 0) atomicCAS(p.status, 0, ZZ_ERR_CAPACITY);
            cp_async_wait<0>();     // stages fetched before the wait
            return;
        }
    }
    if (fused) {
        const int t = len_old;
        new_slot = (p.kind == ZZ_KIND_RETRIEVAL || t < p.S) ? t : p.S + ((t - p.S) % p.W);
        const long long src = ((long long)b * p.n_kv_total + head_list_p[p.kv_head0 + hg]) * HD;
        knew = k_new_p + src;
        vnew = v_new_p + src;
    }

    const int s0 = min(split * p.chunk[b], n);
    const int s1 = (split == nsplit - 1) ? n : min(n, s0 + p.chunk[b]);
    const int nblk = (s1 - s0 + kBlk - 1) / kBlk;              // 16-token blocks of this CTA
    const int my_blocks = (nblk > warp) ? (nblk - warp + kWarps - 1) / kWarps : 0;

    // ---- fused append: the CTA whose range holds the new slot stores the row ----------------
    if (fused && new_slot >= s0 && new_slot < s1 && warp == kWarps - 1) {
        const int c = lane & 15;
        const __nv_bfloat16* src = (lane < 16 ? knew : vnew) + c * 8;
        long long slot_off = (long long)new_slot * HD;
        if (paged)
            slot_off = (long long)tbl[(new_slot >> 7) * p.Hg] * kPageElems + (new_slot & (kPageTokens - 1)) * HD;
        __nv_bfloat16* dst = (lane < 16 ? kbase : vbase) + slot_off + c * 8;
        if (c < HD / 8) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);   // a row has HD / 8 pieces
        if (p.kind == ZZ_KIND_STREAMING && hg == 0 && lane == 0) pos_p[(long long)b * p.ring + new_slot] = len_old;
    }

    // ---- query fragments: rows = the G heads of this KV head ---------------------------
    const int G = p.G;
    const __nv_bfloat16* qb = q_p + ((long long)b * p.q_tok_stride) + (long long)(p.q_head0 + hg * G) * HD;
    uint32_t qa[kKSteps][4];
#pragma unroll
    for (int kk = 0; kk < kKSteps; ++kk) {
        const int d0 = kk * 16 + tig * 2;
        qa[kk][0] = (grp < G) ? *reinterpret_cast<const uint32_t*>(qb + grp * HD + d0) : 0u;
        qa[kk][2] = (grp < G) ? *reinterpret_cast<const uint32_t*>(qb + grp * HD + d0 + 8) : 0u;
        if (HI) {
            qa[kk][1] = (grp + 8 < G) ? *reinterpret_cast<const uint32_t*>(qb + (grp + 8) * HD + d0) : 0u;
            qa[kk][3] = (grp + 8 < G) ? *reinterpret_cast<const uint32_t*>(qb + (grp + 8) * HD + d0 + 8) : 0u;
        } else {
            qa[kk][1] = 0u;
            qa[kk][3] = 0u;
        }
    }

    // ---- per-warp state ------------------------------------------------------------------
    constexpr int NR = HI ? 2 : 1;       // row halves carried
    float o[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};

    // Paged store: lane i holds the page of token block pg0 + i (32 pages = 4096 tokens); a block's
    // page is a shuffle away, the window is reloaded when the warp walks past it.  Blocks start at
    // multiples of 16 tokens (the split plan of a paged cache guarantees it), so a block never
    // straddles a page.  The offset returned maps token t of the block to its row: base + off + t*128.
    const int n_pages = paged ? (sd.cap + kPageTokens - 1) / kPageTokens : 0;
    int pg0 = s0 >> 7;
    int win = (paged && pg0 + lane < n_pages) ? tbl[(pg0 + lane) * p.Hg] : 0;
    auto page_off = [&](int tok0) -> long long {
        if constexpr (!paged) return 0ll;
        const int pg = tok0 >> 7;
        if (pg - pg0 >= 32) {
            pg0 = pg;
            win = (pg0 + lane < n_pages) ? tbl[(pg0 + lane) * p.Hg] : 0;
        }
        const int page = __shfl_sync(0xffffffffu, win, pg - pg0);
        return (long long)page * kPageElems - (long long)pg * kPageTokens * HD;
    };

    // prologue: fill kStages-1 stages
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) {
        if (s < my_blocks && !((pre >> s) & 1u)) {
            const int tok0 = s0 + (warp + s * kWarps) * kBlk;
            const long long po = page_off(tok0);
            load_block<HD>(wbase + s * 2 * kStageBytes, wbase + s * 2 * kStageBytes + kStageBytes, kbase + po, vbase + po,
                       tok0, s1, lane, new_slot, knew, vnew, l2_policy);
        }
        cp_async_commit();
    }

    for (int it = 0; it < my_blocks; ++it) {
        {   // keep the pipeline full
            const int nx = it + kStages - 1;
            if (nx < my_blocks) {
                const int st = nx % kStages;
                const int tok0 = s0 + (warp + nx * kWarps) * kBlk;
                const long long po = page_off(tok0);
                load_block<HD>(wbase + st * 2 * kStageBytes, wbase + st * 2 * kStageBytes + kStageBytes, kbase + po,
                           vbase + po, tok0, s1, lane, new_slot, knew, vnew, l2_policy);
            }
            cp_async_commit();
        }
        cp_async_wait<kStages - 1>();
        __syncwarp();

        const int st = it % kStages;
        const uint32_t sk = wbase + st * 2 * kStageBytes;
        const uint32_t sv = sk + kStageBytes;
        const int tok0 = s0 + (warp + it * kWarps) * kBlk;

        // S = Q K^T for 16 tokens: two 8-token column tiles
        float sc[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < kKSteps; ++kk) {
            const int r = (lane & 7) + ((lane >> 4) << 3);
            const int c = kk * 2 + ((lane >> 3) & 1);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(sk + r * kRowB + ((c ^ (r & 7)) << 4), b0, b1, b2, b3);
            mma_bf16(sc[0], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b0, b1);
            mma_bf16(sc[1], qa[kk][0], qa[kk][1], qa[kk][2], qa[kk][3], b2, b3);
        }

        // online softmax in the log2 domain; mask tokens past the range end
        const int valid = s1 - tok0;   // >= 1
        uint32_t pa[4];
#pragma unroll
        for (int hf = 0; hf < NR; ++hf) {
            float t[4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
                for (int e = 0; e < 2; ++e) t[nt * 2 + e] = sc[nt][hf * 2 + e];
            }
            if (valid < kBlk) {        // the last block of a range (warp-uniform)
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
                    for (int e = 0; e < 2; ++e)
                        if (nt * 8 + tig * 2 + e >= valid) t[nt * 2 + e] = -INFINITY;
                }
            }
            // the scale is positive, so the maximum is taken on the raw scores
            float mx = fmaxf(fmaxf(t[0], t[1]), fmaxf(t[2], t[3]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[hf], mx * p.scale_log2);   // finite: column 0 is always valid
            float ps = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                t[e] = fast_exp2(fmaf(t[e], p.scale_log2, -m_new));
                ps += t[e];
            }
            // the accumulators are rescaled only when some row of the warp raised its maximum
            // (always on the first block, rarely later)
            if (__any_sync(0xffffffffu, m_new > m_run[hf])) {
                const float alpha = fast_exp2(m_run[hf] - m_new);  // 0 on the first block
                l_run[hf] = l_run[hf] * alpha + ps;
#pragma unroll
                for (int i = 0; i < HD / 8; ++i) {
                    o[i][hf * 2 + 0] *= alpha;
                    o[i][hf * 2 + 1] *= alpha;
                }
            } else {
                l_run[hf] += ps;
            }
            m_run[hf] = m_new;
            pa[hf] = pack_bf16(t[0], t[1]);          // tokens 0..7 of the block  (k low)
            pa[2 + hf] = pack_bf16(t[2], t[3]);      // tokens 8..15              (k high)
        }
        if (!HI) { pa[1] = 0u; pa[3] = 0u; }

        // O += P V
#pragma unroll
        for (int nn = 0; nn < kKSteps; ++nn) {
            const int r = (lane & 7) + (((lane >> 3) & 1) << 3);
            const int c = nn * 2 + (lane >> 4);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(sv + r * kRowB + ((c ^ (r & 7)) << 4), b0, b1, b2, b3);
            mma_bf16(o[2 * nn], pa[0], pa[1], pa[2], pa[3], b0, b1);
            mma_bf16(o[2 * nn + 1], pa[0], pa[1], pa[2], pa[3], b2, b3);
        }
        __syncwarp();
    }
    cp_async_wait<0>();
    // everything up to here read only this layer's stores, lengths and the caller's q/k/v
    if (p.gdc_wait) asm volatile("griddepcontrol.wait;" ::: "memory");

    finish_item<kWarps, NR, ColsBf16, HD>(p, smem, &s_is_last, o, m_run, l_run, item, b, hg, nsplit, len_old,
                                      fused && p.bump_len, len_p, out_p, part_o_p, part_ml_p, counters_p, seq_counters_p);
}

}  // namespace

template <bool HI, int kWarps, bool kPaged, int HD>
static cudaError_t setup_one() {
    return cudaFuncSetAttribute(decode_kernel<HI, kWarps, kPaged, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kWarps * kWarpSmem);
}

cudaError_t decode_setup() {
    cudaError_t e = setup_one<false, 4, false, 128>();
    if (e == cudaSuccess) e = setup_one<true, 4, false, 128>();
    if (e == cudaSuccess) e = setup_one<false, 8, false, 128>();
    if (e == cudaSuccess) e = setup_one<true, 8, false, 128>();
    if (e == cudaSuccess) e = setup_one<false, 4, true, 128>();
    if (e == cudaSuccess) e = setup_one<true, 4, true, 128>();
    if (e == cudaSuccess) e = setup_one<false, 8, true, 128>();
    if (e == cudaSuccess) e = setup_one<true, 8, true, 128>();
    if (e == cudaSuccess) e = setup_one<false, 4, false, 64>();
    if (e == cudaSuccess) e = setup_one<true, 4, false, 64>();
    if (e == cudaSuccess) e = setup_one<false, 8, false, 64>();
    if (e == cudaSuccess) e = setup_one<true, 8, false, 64>();
    return e;
}

// overlap != 0: programmatic stream serialization -- the launch may begin while the previous launch
// in the stream is still draining.  Only for launches whose early reads (this layer's stores and
// lengths, the caller's q/k/v) the previous launch cannot have written.  overlap == 2: the launch
// shares nothing at all with the previous one and does not wait for it.  overlap == 3: the kernel
// waits for the previous launch at entry, before it reads anything (always safe; only the launch
// latency overlaps).
cudaError_t launch_decode(const DecodeParams& p, int n_items, int warps, cudaStream_t s, int overlap, int n_layers) {
    if (n_items <= 0) return cudaSuccess;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(n_items, n_layers > 0 ? n_layers : 1);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = warps * kWarpSmem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    DecodeParams pp = p;
    pp.gdc_wait = (overlap == 2) ? 0 : (overlap == 3) ? 2 : 1;
    const bool paged = p.page_table != nullptr && p.kind == ZZ_KIND_RETRIEVAL;
    const bool hi = p.G > 8;
    cudaError_t e;
    if (warps != 4 && warps != 8) return cudaErrorInvalidValue;
    if (p.D != 128 && (p.D != 64 || paged)) return cudaErrorInvalidValue;   // paged stores: head_dim 128 only
#define ZZ_LAUNCH(HI_, W_, PG_) e = cudaLaunchKernelEx(&cfg, decode_kernel<HI_, W_, PG_, 128>, pp)
#define ZZ_LAUNCH64(HI_, W_) e = cudaLaunchKernelEx(&cfg, decode_kernel<HI_, W_, false, 64>, pp)
    if (p.D == 64) {
        if (warps == 8) { if (hi) ZZ_LAUNCH64(true, 8); else ZZ_LAUNCH64(false, 8); }
        else { if (hi) ZZ_LAUNCH64(true, 4); else ZZ_LAUNCH64(false, 4); }
    } else if (warps == 8) {
        if (paged) { if (hi) ZZ_LAUNCH(true, 8, true); else ZZ_LAUNCH(false, 8, true); }
        else { if (hi) ZZ_LAUNCH(true, 8, false); else ZZ_LAUNCH(false, 8, false); }
    } else {
        if (paged) { if (hi) ZZ_LAUNCH(true, 4, true); else ZZ_LAUNCH(false, 4, true); }
        else { if (hi) ZZ_LAUNCH(true, 4, false); else ZZ_LAUNCH(false, 4, false); }
    }
#undef ZZ_LAUNCH
#undef ZZ_LAUNCH64
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace zz
