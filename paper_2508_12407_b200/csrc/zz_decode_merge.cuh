// Pieces shared by the decode kernels (bf16 stores and FP8 retrieval stores): the asynchronous-copy,
// ldmatrix and mma.sync wrappers, and the tail of a work item -- merge of the warps of a CTA, the
// split partials, the length update of a fused or preceding append, and the merge of the splits by
// the last CTA of a (sequence, KV head) to arrive.
#pragma once

#include "zz_common.cuh"

namespace zz {

constexpr int kMaxSplitsSmem = kDecodeSplitSlots;   // merge rows; the host's split limit is below it

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async16_full(uint32_t dst, const void* src, uint64_t policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                            uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1,
                                                  uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// The accumulator tile i (of 16) of a thread holds, for row halves hf = 0, 1 and e = 0, 1, the output
// column col(i, e): the bf16 kernel's tiles are 8 consecutive columns, the FP8 kernel's tiles take
// every other column of a 16-column piece (its V rows are transposed two bytes at a time).
struct ColsBf16 {
    static constexpr bool kAdjacent = true;   // col(i, tig, 1) == col(i, tig, 0) + 1, an even column first
    __device__ __forceinline__ static int col(int i, int tig, int e) { return i * 8 + tig * 2 + e; }
};
struct ColsFp8 {
    static constexpr bool kAdjacent = false;
    __device__ __forceinline__ static int col(int i, int tig, int e) { return (i >> 1) * 16 + tig * 4 + e * 2 + (i & 1); }
};

template <int kWarps, int HD>
__device__ __forceinline__ void finish_item_tail(const DecodeParams& p, unsigned char* smem, int* s_is_last_p, int item,
                                                 int b, int hg, int nsplit, int len_old, bool advance_len,
                                                 int* len_p, __nv_bfloat16* out_p, float* part_o_p, float* part_ml_p,
                                                 unsigned int* counters_p, unsigned int* seq_counters_p);

// Everything after a CTA's main loop.  `advance_len`: this launch makes the sequence one token longer
// (the append fused into it, or the quantising append that ran just before it) and is the layer's last.
template <int kWarps, int NR, class Cols, int HD = kD>
__device__ __forceinline__ void finish_item(const DecodeParams& p, unsigned char* smem, int* s_is_last_p,
                                            float (&o)[HD / 8][4], float (&m_run)[2], float (&l_run)[2], int item,
                                            int b, int hg, int nsplit, int len_old, bool advance_len,
                                            int* len_p, __nv_bfloat16* out_p, float* part_o_p, float* part_ml_p,
                                            unsigned int* counters_p, unsigned int* seq_counters_p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = lane >> 2, tig = lane & 3;
    const int G = p.G;
    // ---- merge the warps of this CTA ---------------------------------------------------------
#pragma unroll
    for (int hf = 0; hf < NR; ++hf) {
        l_run[hf] += __shfl_xor_sync(0xffffffffu, l_run[hf], 1);
        l_run[hf] += __shfl_xor_sync(0xffffffffu, l_run[hf], 2);
    }
    __syncthreads();   // every warp is done with its pipeline memory
    float* sm_o = reinterpret_cast<float*>(smem);                  // [kWarps][16][128]
    float* sm_ml = sm_o + kWarps * 16 * HD;                        // [kWarps][16][2]
#pragma unroll
    for (int hf = 0; hf < NR; ++hf) {
        const int row = grp + hf * 8;
        if (row < G) {
#pragma unroll
            for (int i = 0; i < HD / 8; ++i) {
                if constexpr (Cols::kAdjacent) {
                    *reinterpret_cast<float2*>(sm_o + (warp * 16 + row) * HD + Cols::col(i, tig, 0)) =
                        make_float2(o[i][hf * 2], o[i][hf * 2 + 1]);
                } else {
                    sm_o[(warp * 16 + row) * HD + Cols::col(i, tig, 0)] = o[i][hf * 2];
                    sm_o[(warp * 16 + row) * HD + Cols::col(i, tig, 1)] = o[i][hf * 2 + 1];
                }
            }
            if (tig == 0) {
                sm_ml[(warp * 16 + row) * 2 + 0] = m_run[hf];
                sm_ml[(warp * 16 + row) * 2 + 1] = l_run[hf];
            }
        }
    }
    __syncthreads();
    finish_item_tail<kWarps, HD>(p, smem, s_is_last_p, item, b, hg, nsplit, len_old, advance_len, len_p, out_p, part_o_p,
                                 part_ml_p, counters_p, seq_counters_p);
}

// The part of the tail that starts from the warps' results staged in shared memory (sm_o [kWarps][16][HD]
// fp32 rows of the group's query heads, then sm_ml [kWarps][16][2] = running maximum and sum), all warps
// past a __syncthreads.
template <int kWarps, int HD>
__device__ __forceinline__ void finish_item_tail(const DecodeParams& p, unsigned char* smem, int* s_is_last_p, int item,
                                                 int b, int hg, int nsplit, int len_old, bool advance_len,
                                                 int* len_p, __nv_bfloat16* out_p, float* part_o_p, float* part_ml_p,
                                                 unsigned int* counters_p, unsigned int* seq_counters_p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.G;
    int& s_is_last = *s_is_last_p;
    float* sm_o = reinterpret_cast<float*>(smem);                  // [kWarps][16][HD]
    float* sm_ml = sm_o + kWarps * 16 * HD;                        // [kWarps][16][2]

    const long long pair = (long long)b * p.Hg + hg;
    __nv_bfloat16* outb = out_p + ((long long)b * p.q_tok_stride) + (long long)(p.q_head0 + hg * G) * HD;
    for (int idx = threadIdx.x; idx < G * HD; idx += kWarps * 32) {
        const int row = idx / HD, d = idx % HD;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_ml[(w * 16 + row) * 2]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float mw = sm_ml[(w * 16 + row) * 2];
            const float f = (mw == -INFINITY) ? 0.f : fast_exp2(mw - M);
            L += f * sm_ml[(w * 16 + row) * 2 + 1];
            acc += f * sm_o[(w * 16 + row) * HD + d];
        }
        if (nsplit == 1) {
            outb[row * HD + d] = __float2bfloat16_rn(acc / L);
        } else {
            const long long po = (long long)item * G + row;   // partials are indexed by work item
            part_o_p[po * HD + d] = acc;
            if (d == 0) {
                part_ml_p[po * 2 + 0] = M;
                part_ml_p[po * 2 + 1] = L;
            }
        }
    }
    if (advance_len) {
        // every CTA of the sequence has read the old length by the time it gets here; the last
        // one to arrive publishes the new length
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned int all = (unsigned int)(nsplit * p.Hg);
            const unsigned int prev = atomicAdd(seq_counters_p + b, 1u);
            if (prev == all - 1) {
                len_p[b] = len_old + 1;
                seq_counters_p[b] = 0u;
            }
        }
    }
    if (nsplit == 1) return;

    // ---- last CTA of this (sequence, head) merges the splits -----------------------------------
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int prev = atomicAdd(counters_p + pair, 1u);
        s_is_last = (prev == (unsigned int)(nsplit - 1));
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    // Merge of the splits in (about) one memory round trip: thread (row, 4 dims) first issues the
    // float4 loads of every split's partial output, then the (max, sum) pairs are turned into
    // per-split factors through shared memory while those loads are in flight.
    float* sm_m = reinterpret_cast<float*>(smem);            // [16][128] running max per split
    float* sm_f = sm_m + 16 * kMaxSplitsSmem;                // [16][128] sum, then factor
    constexpr int kRound = 40;                               // splits whose partials are held at once (one round for the usual 37 of a 32K store)
    for (int row0 = 0; row0 < G; row0 += kWarps) {
        const int row = row0 + warp;                         // this warp's row (4 dims per lane; half the lanes at head_dim 64)
        const bool row_ok = row < G && lane * 4 < HD;
        // split s of this (sequence, head) is work item item0 + s * Hg
        const long long item0 = (long long)p.split_start[b] * p.Hg + hg;
        const float* pbase = part_o_p + (item0 * G + (row_ok ? row : 0)) * HD + lane * 4;
        const long long sstride = (long long)p.Hg * G * HD;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sb = 0; sb < nsplit; sb += kRound) {
            float4 v[kRound];
#pragma unroll
            for (int u = 0; u < kRound; ++u)
                v[u] = (row_ok && sb + u < nsplit) ? __ldcg(reinterpret_cast<const float4*>(pbase + (sb + u) * sstride))
                                                   : make_float4(0.f, 0.f, 0.f, 0.f);
            if (sb == 0) {
                for (int i = threadIdx.x; i < nsplit * kWarps; i += blockDim.x) {
                    const int s = i / kWarps, r = row0 + i % kWarps;
                    if (r < G) {
                        const long long po = (item0 + (long long)s * p.Hg) * G + r;
                        const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_ml_p + po * 2));
                        sm_m[r * kMaxSplitsSmem + s] = ml.x;
                        sm_f[r * kMaxSplitsSmem + s] = ml.y;
                    }
                }
                __syncthreads();
                if (row < G) {
                    float M = -INFINITY;
                    for (int s = lane; s < nsplit; s += 32) M = fmaxf(M, sm_m[row * kMaxSplitsSmem + s]);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
                    float L = 0.f;
                    for (int s = lane; s < nsplit; s += 32) {
                        const float ms = sm_m[row * kMaxSplitsSmem + s];
                        const float f = (ms == -INFINITY) ? 0.f : fast_exp2(ms - M);
                        L += f * sm_f[row * kMaxSplitsSmem + s];
                        sm_f[row * kMaxSplitsSmem + s] = f;
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
                    if (lane == 0) sm_m[row * kMaxSplitsSmem + kMaxSplitsSmem - 1] = 1.f / L;  // slot no split uses
                }
                __syncwarp();
            }
#pragma unroll
            for (int u = 0; u < kRound; ++u) {
                if (row_ok && sb + u < nsplit) {
                    const float f = sm_f[row * kMaxSplitsSmem + sb + u];
                    acc.x += f * v[u].x; acc.y += f * v[u].y; acc.z += f * v[u].z; acc.w += f * v[u].w;
                }
            }
        }
        if (row_ok) {
            const float inv = sm_m[row * kMaxSplitsSmem + kMaxSplitsSmem - 1];
            uint2 w;
            w.x = pack_bf16(acc.x * inv, acc.y * inv);
            w.y = pack_bf16(acc.z * inv, acc.w * inv);
            *reinterpret_cast<uint2*>(outb + row * HD + lane * 4) = w;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) counters_p[pair] = 0u;
}

}  // namespace zz
