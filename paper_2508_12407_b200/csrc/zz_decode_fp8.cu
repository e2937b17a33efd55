// FP8 retrieval stores: the quantising append, the decode kernel over FP8 rows, and the expansion of
// an FP8 store to bf16 rows for the prefill kernel.
//
// A stored row (one token, one KV head) is 128 E4M3 codes plus one scale byte e standing for 2^(e-127):
// the smallest power of two that brings the row's largest magnitude to at most 448, the largest E4M3
// number.  The stored value is code * 2^(e-127) exactly, so the store halves the bytes a decode step
// has to read (258 instead of 512 per token, head and K/V pair).
//
// Decode: same split-sequence plan, work items and merge as the bf16 kernel.  The codes convert to
// f16 exactly (one cvt per pair), so QK^T and PV run as f16 mma.sync tiles:
//   * the query rows are scaled by a power of two per row so that they convert to f16 without loss of
//     range; that factor, the softmax scale and the K scale of each token are applied to the fp32
//     scores;
//   * the V scale of each token multiplies its probability before that is rounded to f16, relative to
//     the largest V scale the warp has met so far (the accumulators are rescaled when it grows), so the
//     f16 operand never overflows and rows with tiny scales simply contribute little.
// Groups of up to eight query heads run decode_fp8t_kernel, which computes both products transposed
// (see there); larger groups run decode_fp8_kernel.
// An 8-bit row is 128 bytes: ldmatrix moves it as 16-bit units, which puts four consecutive dims of a
// token into a thread's register for K (the query fragments are loaded in the matching order) and two
// dims of two consecutive tokens for V (a byte permute separates them; an accumulator tile therefore
// holds every other column of a 16-column piece, see ColsFp8).
#include <cuda_fp16.h>

#include <cstring>

#include "zz_decode_merge.cuh"

namespace zz {

namespace {

constexpr int kBlk = 16;                          // tokens per warp step
constexpr int kStagesF8 = 4;
constexpr int kCodeBytes = kBlk * kD;             // 2 KiB of K codes (and as much of V codes) per stage
constexpr int kStageF8 = 2 * kCodeBytes + 128;    // + 16 K scale bytes, 16 V scale bytes, padding
constexpr int kWarpSmemF8 = kStagesF8 * kStageF8; // 16896 B per warp: 4 warps 66 KiB (three CTAs per SM), 8 warps 132 KiB

__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two E4M3 codes (low byte first) -> f16x2, exact
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_codes) {
    uint32_t r;
    const unsigned short x = (unsigned short)two_codes;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;\n" : "=r"(r) : "h"(x));
    return r;
}
// the four codes of a 32-bit register -> two f16x2 registers (codes 0, 1 and codes 2, 3)
__device__ __forceinline__ void e4m3x4_to_f16x2x2(uint32_t four_codes, uint32_t& lo, uint32_t& hi) {
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\t"
        "cvt.rn.f16x2.e4m3x2 %0, a;\n\tcvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
        : "=r"(lo), "=r"(hi)
        : "r"(four_codes));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// two floats -> two E4M3 codes (round to nearest even, saturating), low byte = lo
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {
    unsigned short r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;\n" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float pow2_of_byte(int e) { return __uint_as_float((uint32_t)e << 23); }   // 2^(e-127), e in 0..254

// scale byte of a row whose largest bf16 magnitude has the bit pattern amax (sign cleared)
__device__ __forceinline__ int fp8_scale_byte(uint32_t amax) {
    int e = (int)(amax >> 7) - 8 + (((amax & 0x7Fu) > 0x60u) ? 1 : 0);
    return e < 1 ? 1 : e;
}

// ---------------------------------------------------------------------------------------------
// Quantising append.  Sixteen consecutive threads own one row (8 values each) of K and of V.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) quant_append_kernel(const QuantAppendParams p) {
    const int b = blockIdx.y;
    const int li = p.layer_ids ? p.layer_ids[blockIdx.z] : p.layer;
    const SeqDesc sd = p.desc_table[(long long)li * p.B + b];
    const int P = p.len[(long long)li * p.B + b];
    const int C = p.layer_ids ? 1 : p.n_new[b];
    // room?  (the host has checked; a launch replayed from a graph checks for itself)
    if (P + C > sd.cap) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(p.status, 0, ZZ_ERR_CAPACITY);
        return;
    }
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const bool active = idx < (long long)C * p.nR * 16;
    const int piece = (int)(idx & 15);
    const long long r = idx >> 4;
    const int hi = active ? (int)(r % p.nR) : 0;
    const int i = active ? (int)(r / p.nR) : 0;
    const int src_head = p.head_list[(long long)li * p.Hkv + hi];
    long long src;
    if (p.layer_ids) src = (((long long)li * p.B + b) * p.Hkv + src_head) * kD + piece * 8;
    else src = ((long long)(p.tok_off[b] + i) * p.Hkv + src_head) * kD + piece * 8;
    const int cap16 = fp8_cap16(sd.cap);
    unsigned char* const kcodes = p.arena + 2 * sd.k_off[ZZ_KIND_RETRIEVAL];
    unsigned char* const vcodes = p.arena + 2 * sd.v_off[ZZ_KIND_RETRIEVAL];
    unsigned char* const kscale = p.arena + fp8_kscale_byte_off(sd.v_off[ZZ_KIND_RETRIEVAL], p.nR, sd.cap);
    unsigned char* const vscale = kscale + (long long)p.nR * cap16;
    const long long slot = (long long)P + i;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        uint4 x = make_uint4(0u, 0u, 0u, 0u);
        if (active) x = *reinterpret_cast<const uint4*>((which ? p.v_new : p.k_new) + src);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
        uint32_t amax = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            amax = max(amax, w[j] & 0x7FFFu);
            amax = max(amax, (w[j] >> 16) & 0x7FFFu);
        }
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, o, 16));
        const int e = fp8_scale_byte(amax);
        const float inv = pow2_of_byte(254 - e);      // 2^(127 - e); e <= 247 for finite bf16 input
        uint32_t codes[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float a0 = __uint_as_float(w[2 * j] << 16) * inv, a1 = __uint_as_float(w[2 * j] & 0xFFFF0000u) * inv;
            const float a2 = __uint_as_float(w[2 * j + 1] << 16) * inv, a3 = __uint_as_float(w[2 * j + 1] & 0xFFFF0000u) * inv;
            codes[j] = f32x2_to_e4m3x2(a0, a1) | (f32x2_to_e4m3x2(a2, a3) << 16);
        }
        if (active) {
            unsigned char* dst = (which ? vcodes : kcodes) + ((long long)hi * sd.cap + slot) * kD + piece * 8;
            *reinterpret_cast<uint2*>(dst) = make_uint2(codes[0], codes[1]);
            if (piece == 0) (which ? vscale : kscale)[(long long)hi * cap16 + slot] = (unsigned char)e;
        }
    }
}

// FP8 rows -> bf16 rows (exact: four significant bits and a power-of-two scale).
__global__ void __launch_bounds__(256) dequant_kernel(const DequantParams p) {
    const int b = blockIdx.y;
    const int P = p.len[b];
    const SeqDesc s = p.src[b], d = p.dst[b];
    const int cap16 = fp8_cap16(s.cap);
    const unsigned char* const kscale = p.arena + fp8_kscale_byte_off(s.v_off[ZZ_KIND_RETRIEVAL], p.nR, s.cap);
    const unsigned char* const vscale = kscale + (long long)p.nR * cap16;
    const long long total = (long long)P * p.nR * 16;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int piece = (int)(idx & 15);
        const long long r = idx >> 4;
        const int hi = (int)(r / P);
        const long long slot = r % P;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            const unsigned char* codes = p.arena + 2 * (which ? s.v_off : s.k_off)[ZZ_KIND_RETRIEVAL] +
                                         ((long long)hi * s.cap + slot) * kD + piece * 8;
            const uint2 c = *reinterpret_cast<const uint2*>(codes);
            const float sc = pow2_of_byte((which ? vscale : kscale)[(long long)hi * cap16 + slot]);
            const uint32_t cw[2] = {c.x, c.y};
            uint32_t out[4];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const uint32_t h0 = e4m3x2_to_f16x2(cw[j] & 0xFFFFu), h1 = e4m3x2_to_f16x2(cw[j] >> 16);
                const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&h0));
                const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&h1));
                out[2 * j] = pack_bf16(f0.x * sc, f0.y * sc);
                out[2 * j + 1] = pack_bf16(f1.x * sc, f1.y * sc);
            }
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.arena) + (which ? d.v_off : d.k_off)[ZZ_KIND_RETRIEVAL] +
                                 ((long long)hi * d.cap + slot) * kD + piece * 8;
            *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Decode over FP8 rows.
// ---------------------------------------------------------------------------------------------
// One 16-token block into a stage: K codes at +0, V codes at +2048 (row r, 16-byte piece c at
// r * 128 + ((c ^ (r & 7)) * 16)), the 16 K scale bytes at +4096, the 16 V scale bytes at +4112.
// Blocks start at multiples of 16 tokens (the split plan of an FP8 cache sees to it), so the scale
// bytes of a block are one aligned 16-byte piece.
__device__ __forceinline__ void load_block_fp8(uint32_t stage, const unsigned char* kc, const unsigned char* vc,
                                               const unsigned char* ks, const unsigned char* vs, int tok0, int tok_end,
                                               int lane, uint64_t policy) {
    const int c = lane & 7;
    if (tok0 + kBlk <= tok_end) {
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int r = it * 4 + (lane >> 3);
            const long long off = (long long)(tok0 + r) * kD + c * 16;
            const uint32_t so = r * kD + ((c ^ (r & 7)) << 4);
            cp_async16_full(stage + so, kc + off, policy);
            cp_async16_full(stage + kCodeBytes + so, vc + off, policy);
        }
    } else {
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int r = it * 4 + (lane >> 3);
            const int ok = tok0 + r < tok_end;
            const long long off = (long long)(ok ? tok0 + r : tok0) * kD + c * 16;
            const uint32_t so = r * kD + ((c ^ (r & 7)) << 4);
            cp_async16(stage + so, kc + off, ok ? 16 : 0);
            cp_async16(stage + kCodeBytes + so, vc + off, ok ? 16 : 0);
        }
    }
    if (lane < 2) cp_async16(stage + 2 * kCodeBytes + lane * 16, (lane ? vs : ks) + tok0, 16);
}

// Twice the tokens per byte make this kernel bound by instruction issue rather than by HBM, and its
// chains of dependent steps are long: twelve warps per SM (168 registers, four stages) measured 7-8 %
// faster than eight (225 registers, six stages).
template <bool HI, int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 12 / kWarps) decode_fp8_kernel(const DecodeParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ int s_is_last;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = lane >> 2, tig = lane & 3;

    // programmatic dependent launch, as in the bf16 kernel
    if (p.gdc_wait == 2) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int li = p.layer_ids ? p.layer_ids[blockIdx.y] : 0;
    int* const len_p = p.len + (long long)li * p.st_len;
    const __nv_bfloat16* const q_p = p.q + (long long)li * p.st_q;
    __nv_bfloat16* const out_p = p.out + (long long)li * p.st_q;
    unsigned int* const counters_p = p.counters + (long long)li * p.st_cnt;
    unsigned int* const seq_counters_p = p.seq_counters + (long long)li * p.st_cnt;
    float* const part_o_p = p.part_o + (long long)li * p.st_part * kD;
    float* const part_ml_p = p.part_ml + (long long)li * p.st_part * 2;

    const int item = blockIdx.x;
    int b = 0;
    while (b + 1 < p.B && item >= p.split_start[b + 1] * p.Hg) ++b;
    const int local = item - p.split_start[b] * p.Hg;
    const int hg = local % p.Hg;
    const int split = local / p.Hg;
    const int nsplit = p.split_start[b + 1] - p.split_start[b];
    if (nsplit > p.max_splits || p.max_splits > kDecodeMaxSplits) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, ZZ_ERR_UNSUPPORTED);
        return;
    }

    const int len_old = len_p[b];
    const SeqDesc sd = p.layer_ids ? p.desc_table[(long long)li * p.B + b] : p.sd[b];
    if (p.appended && len_old >= sd.cap) {
        // a replayed step without room: the append before this launch stored nothing either
        if (threadIdx.x == 0) atomicCAS(p.status, 0, ZZ_ERR_CAPACITY);
        return;
    }
    const int n = len_old + (p.appended ? 1 : 0);
    const int cap16 = fp8_cap16(sd.cap);
    const unsigned char* const arena8 = reinterpret_cast<const unsigned char*>(p.arena);
    const unsigned char* const kc = arena8 + 2 * sd.k_off[ZZ_KIND_RETRIEVAL] + (long long)hg * sd.cap * kD;
    const unsigned char* const vc = arena8 + 2 * sd.v_off[ZZ_KIND_RETRIEVAL] + (long long)hg * sd.cap * kD;
    const unsigned char* const ks = arena8 + fp8_kscale_byte_off(sd.v_off[ZZ_KIND_RETRIEVAL], p.Hg, sd.cap) + (long long)hg * cap16;
    const unsigned char* const vs = ks + (long long)p.Hg * cap16;

    const int s0 = min(split * p.chunk[b], n);
    const int s1 = (split == nsplit - 1) ? n : min(n, s0 + p.chunk[b]);
    const int nblk = (s1 - s0 + kBlk - 1) / kBlk;
    const int my_blocks = (nblk > warp) ? (nblk - warp + kWarps - 1) / kWarps : 0;

    // ---- query fragments: each row scaled by a power of two into f16's range --------------------
    // thread (grp, tig) holds dims 16 kk + 4 tig + {0, 1} (a0 / a1) and + {2, 3} (a2 / a3) of rows grp and grp + 8:
    // the order in which ldmatrix hands out the bytes of an 8-bit K row
    const int G = p.G;
    constexpr int NR = HI ? 2 : 1;
    const __nv_bfloat16* qb = q_p + ((long long)b * p.q_tok_stride) + (long long)(p.q_head0 + hg * G) * kD;
    uint32_t qa[8][4];
    float qmul[2] = {0.f, 0.f};
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        if (hf >= NR) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) { qa[kk][hf] = 0u; qa[kk][2 + hf] = 0u; }
            continue;
        }
        const int row = grp + hf * 8;
        uint2 raw[8];
        uint32_t amax = 0;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            raw[kk] = (row < G) ? *reinterpret_cast<const uint2*>(qb + row * kD + kk * 16 + tig * 4) : make_uint2(0u, 0u);
            amax = max(max(amax, raw[kk].x & 0x7FFFu), max((raw[kk].x >> 16) & 0x7FFFu, max(raw[kk].y & 0x7FFFu, (raw[kk].y >> 16) & 0x7FFFu)));
        }
        amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
        int kq = (int)(amax >> 7);                    // exponent field of the row's largest magnitude
        kq = kq > 253 ? 253 : kq;
        const float down = pow2_of_byte(254 - kq);    // 2^(127 - kq): the row's largest magnitude lands in [1, 4)
        qmul[hf] = p.scale_log2 * pow2_of_byte(kq);   // kq = 0 (an all-zero row): 0
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            qa[kk][hf] = pack_f16(__uint_as_float(raw[kk].x << 16) * down, __uint_as_float(raw[kk].x & 0xFFFF0000u) * down);
            qa[kk][2 + hf] = pack_f16(__uint_as_float(raw[kk].y << 16) * down, __uint_as_float(raw[kk].y & 0xFFFF0000u) * down);
        }
    }

    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};
    int eref = 0;                                     // largest V scale byte met so far: o is in units of 2^(eref-127)

    const uint32_t wbase = smem_u32(smem) + warp * kWarpSmemF8;
    uint64_t l2_policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(l2_policy));

#pragma unroll
    for (int s = 0; s < kStagesF8 - 1; ++s) {
        if (s < my_blocks) {
            const int tok0 = s0 + (warp + s * kWarps) * kBlk;
            load_block_fp8(wbase + s * kStageF8, kc, vc, ks, vs, tok0, s1, lane, l2_policy);
        }
        cp_async_commit();
    }

    for (int it = 0; it < my_blocks; ++it) {
        {
            const int nx = it + kStagesF8 - 1;
            if (nx < my_blocks) {
                const int tok0 = s0 + (warp + nx * kWarps) * kBlk;
                load_block_fp8(wbase + (nx % kStagesF8) * kStageF8, kc, vc, ks, vs, tok0, s1, lane, l2_policy);
            }
            cp_async_commit();
        }
        cp_async_wait<kStagesF8 - 1>();
        __syncwarp();

        const uint32_t sk = wbase + (it % kStagesF8) * kStageF8;
        const uint32_t sv = sk + kCodeBytes;
        const int tok0 = s0 + (warp + it * kWarps) * kBlk;
        const int valid = s1 - tok0;   // >= 1

        // scale bytes of this thread's four tokens: 2 tig, 2 tig + 1, 8 + 2 tig, 9 + 2 tig
        uint32_t kb01, kb89, vb01, vb89;
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(kb01) : "r"(sk + 2 * kCodeBytes + 2 * tig));
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(kb89) : "r"(sk + 2 * kCodeBytes + 8 + 2 * tig));
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(vb01) : "r"(sk + 2 * kCodeBytes + 16 + 2 * tig));
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(vb89) : "r"(sk + 2 * kCodeBytes + 24 + 2 * tig));
        int kbyte[4] = {(int)(kb01 & 0xFF), (int)(kb01 >> 8), (int)(kb89 & 0xFF), (int)(kb89 >> 8)};
        int vbyte[4] = {(int)(vb01 & 0xFF), (int)(vb01 >> 8), (int)(vb89 & 0xFF), (int)(vb89 >> 8)};
        if (valid < kBlk) {            // tokens past the range end carry no scale
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if ((j >> 1) * 8 + tig * 2 + (j & 1) >= valid) { kbyte[j] = 0; vbyte[j] = 0; }
        }

        // S = Q K^T (raw: codes times scaled query)
        float sc[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i) { sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f; }
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
            const int r = (lane & 7) + (((lane >> 3) & 1) << 3);
            const int c = pc * 2 + (lane >> 4);
            uint32_t m0, m1, m2, m3, b0, b1;
            ldmatrix_x4(sk + r * kD + ((c ^ (r & 7)) << 4), m0, m1, m2, m3);
            e4m3x4_to_f16x2x2(m0, b0, b1);
            mma_f16(sc[0], qa[2 * pc][0], qa[2 * pc][1], qa[2 * pc][2], qa[2 * pc][3], b0, b1);
            e4m3x4_to_f16x2x2(m1, b0, b1);
            mma_f16(sc[1], qa[2 * pc][0], qa[2 * pc][1], qa[2 * pc][2], qa[2 * pc][3], b0, b1);
            e4m3x4_to_f16x2x2(m2, b0, b1);
            mma_f16(sc[0], qa[2 * pc + 1][0], qa[2 * pc + 1][1], qa[2 * pc + 1][2], qa[2 * pc + 1][3], b0, b1);
            e4m3x4_to_f16x2x2(m3, b0, b1);
            mma_f16(sc[1], qa[2 * pc + 1][0], qa[2 * pc + 1][1], qa[2 * pc + 1][2], qa[2 * pc + 1][3], b0, b1);
        }

        // the block's largest V scale: the accumulators move to it when it grows (rare after the first block)
        int vmax = max(max(vbyte[0], vbyte[1]), max(vbyte[2], vbyte[3]));
        vmax = max(vmax, __shfl_xor_sync(0xffffffffu, vmax, 1));
        vmax = max(vmax, __shfl_xor_sync(0xffffffffu, vmax, 2));
        if (vmax > eref) {             // warp-uniform: every group of four lanes sees the same 16 tokens
            const float f = pow2_of_byte(max(eref - vmax + 127, 0));
#pragma unroll
            for (int i = 0; i < 16; ++i) { o[i][0] *= f; o[i][1] *= f; o[i][2] *= f; o[i][3] *= f; }
            eref = vmax;
        }
        float vf[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) vf[j] = pow2_of_byte(max(vbyte[j] - eref + 127, 0));

        uint32_t pa[4];
#pragma unroll
        for (int hf = 0; hf < NR; ++hf) {
            float t[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) t[j] = sc[j >> 1][hf * 2 + (j & 1)] * (qmul[hf] * pow2_of_byte(kbyte[j]));
            if (valid < kBlk) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if ((j >> 1) * 8 + tig * 2 + (j & 1) >= valid) t[j] = -INFINITY;
            }
            float mx = fmaxf(fmaxf(t[0], t[1]), fmaxf(t[2], t[3]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[hf], mx);       // finite: token 0 of a block is always valid
            float ps = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                t[j] = fast_exp2(t[j] - m_new);
                ps += t[j];
            }
            if (__any_sync(0xffffffffu, m_new > m_run[hf])) {
                const float alpha = fast_exp2(m_run[hf] - m_new);
                l_run[hf] = l_run[hf] * alpha + ps;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    o[i][hf * 2 + 0] *= alpha;
                    o[i][hf * 2 + 1] *= alpha;
                }
            } else {
                l_run[hf] += ps;
            }
            m_run[hf] = m_new;
            pa[hf] = pack_f16(t[0] * vf[0], t[1] * vf[1]);        // tokens 0..7 of the block
            pa[2 + hf] = pack_f16(t[2] * vf[2], t[3] * vf[3]);    // tokens 8..15
        }
        if (!HI) { pa[1] = 0u; pa[3] = 0u; }

        // O += P V: a transposed 16-bit unit holds dims (2 grp, 2 grp + 1) of tokens 2 tig (low half)
        // and 2 tig + 1 (high half); the permute puts the two tokens of each dim side by side
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
            const int r = (lane & 7) + (((lane >> 3) & 1) << 3);
            const int c = pc * 2 + (lane >> 4);
            uint32_t m0, m1, m2, m3;
            ldmatrix_x4_trans(sv + r * kD + ((c ^ (r & 7)) << 4), m0, m1, m2, m3);
            uint32_t e0, o0, e1, o1;
            e4m3x4_to_f16x2x2(__byte_perm(m0, 0u, 0x3120), e0, o0);
            e4m3x4_to_f16x2x2(__byte_perm(m1, 0u, 0x3120), e1, o1);
            mma_f16(o[4 * pc + 0], pa[0], pa[1], pa[2], pa[3], e0, e1);
            mma_f16(o[4 * pc + 1], pa[0], pa[1], pa[2], pa[3], o0, o1);
            e4m3x4_to_f16x2x2(__byte_perm(m2, 0u, 0x3120), e0, o0);
            e4m3x4_to_f16x2x2(__byte_perm(m3, 0u, 0x3120), e1, o1);
            mma_f16(o[4 * pc + 2], pa[0], pa[1], pa[2], pa[3], e0, e1);
            mma_f16(o[4 * pc + 3], pa[0], pa[1], pa[2], pa[3], o0, o1);
        }
        __syncwarp();
    }
    cp_async_wait<0>();
    if (p.gdc_wait) asm volatile("griddepcontrol.wait;" ::: "memory");

    // back to plain units before the warps are merged
    {
        const float f = pow2_of_byte(eref);
#pragma unroll
        for (int i = 0; i < 16; ++i) { o[i][0] *= f; o[i][1] *= f; o[i][2] *= f; o[i][3] *= f; }
    }
    finish_item<kWarps, NR, ColsFp8>(p, smem, &s_is_last, o, m_run, l_run, item, b, hg, nsplit, len_old,
                                     p.appended && p.bump_len, len_p, out_p, part_o_p, part_ml_p, counters_p, seq_counters_p);
}


// ---------------------------------------------------------------------------------------------
// The same decode step with the products transposed, for groups of up to eight query heads.
//   S^T = K Q^T:  tokens are the 16 rows of the MMA tile, the group's query heads its 8 columns;
//   O^T = V^T P^T: 16 head dims are the rows, the query heads the columns, the block's 16 tokens the
//   contraction.
// A 16 x 8 tile wastes nothing on a group of eight (or four) heads, where the untransposed kernel
// fills at most half of its 16 query rows: half the MMAs, half the accumulator registers (32), half
// the query registers, and with them room for more warps per SM, which is what this issue-bound kernel
// needs.  The probabilities come out of the first product with tokens along the rows and are needed
// with tokens along the contraction: one movmatrix per 8 x 8 block transposes them.
// Thread (grp, tig) of a warp holds, per 16-token block: scores of tokens grp and grp + 8 for heads
// 2 tig and 2 tig + 1; its accumulator tile c holds dims 16 c + 2 grp (+ 1) of those two heads.
// ---------------------------------------------------------------------------------------------
constexpr int kStagesT = 4;
constexpr int kWarpSmemT = kStagesT * kStageF8;   // 16896 B per warp: 4 warps 66 KiB (three CTAs per SM; four CTAs of
                                                  // three stages at 128 registers timed the same and spilled in the merge)

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t r;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(r) : "r"(x));
    return r;
}

template <int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 12 / kWarps) decode_fp8t_kernel(const DecodeParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ int s_is_last;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = lane >> 2, tig = lane & 3;

    if (p.gdc_wait == 2) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int li = p.layer_ids ? p.layer_ids[blockIdx.y] : 0;
    int* const len_p = p.len + (long long)li * p.st_len;
    const __nv_bfloat16* const q_p = p.q + (long long)li * p.st_q;
    __nv_bfloat16* const out_p = p.out + (long long)li * p.st_q;
    unsigned int* const counters_p = p.counters + (long long)li * p.st_cnt;
    unsigned int* const seq_counters_p = p.seq_counters + (long long)li * p.st_cnt;
    float* const part_o_p = p.part_o + (long long)li * p.st_part * kD;
    float* const part_ml_p = p.part_ml + (long long)li * p.st_part * 2;

    const int item = blockIdx.x;
    int b = 0;
    while (b + 1 < p.B && item >= p.split_start[b + 1] * p.Hg) ++b;
    const int local = item - p.split_start[b] * p.Hg;
    const int hg = local % p.Hg;
    const int split = local / p.Hg;
    const int nsplit = p.split_start[b + 1] - p.split_start[b];
    if (nsplit > p.max_splits || p.max_splits > kDecodeMaxSplits) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, ZZ_ERR_UNSUPPORTED);
        return;
    }
    const int len_old = len_p[b];
    const SeqDesc sd = p.layer_ids ? p.desc_table[(long long)li * p.B + b] : p.sd[b];
    if (p.appended && len_old >= sd.cap) {
        if (threadIdx.x == 0) atomicCAS(p.status, 0, ZZ_ERR_CAPACITY);
        return;
    }
    const int n = len_old + (p.appended ? 1 : 0);
    const int cap16 = fp8_cap16(sd.cap);
    const unsigned char* const arena8 = reinterpret_cast<const unsigned char*>(p.arena);
    const unsigned char* const kc = arena8 + 2 * sd.k_off[ZZ_KIND_RETRIEVAL] + (long long)hg * sd.cap * kD;
    const unsigned char* const vc = arena8 + 2 * sd.v_off[ZZ_KIND_RETRIEVAL] + (long long)hg * sd.cap * kD;
    const unsigned char* const ks = arena8 + fp8_kscale_byte_off(sd.v_off[ZZ_KIND_RETRIEVAL], p.Hg, sd.cap) + (long long)hg * cap16;
    const unsigned char* const vs = ks + (long long)p.Hg * cap16;

    const int s0 = min(split * p.chunk[b], n);
    const int s1 = (split == nsplit - 1) ? n : min(n, s0 + p.chunk[b]);
    const int nblk = (s1 - s0 + kBlk - 1) / kBlk;
    const int my_blocks = (nblk > warp) ? (nblk - warp + kWarps - 1) / kWarps : 0;

    // ---- query fragments (B operand of S^T = K Q^T): head grp, dims 16 kk + 4 tig + {0, 1} and + {2, 3},
    // each row scaled by a power of two into f16's range ----------------------------------------------
    const int G = p.G;
    const __nv_bfloat16* qb = q_p + ((long long)b * p.q_tok_stride) + (long long)(p.q_head0 + hg * G) * kD;
    uint32_t qf[8][2];
    float qmul[2];
    {
        uint2 raw[8];
        uint32_t amax = 0;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            raw[kk] = (grp < G) ? *reinterpret_cast<const uint2*>(qb + grp * kD + kk * 16 + tig * 4) : make_uint2(0u, 0u);
            amax = max(max(amax, raw[kk].x & 0x7FFFu), max((raw[kk].x >> 16) & 0x7FFFu, max(raw[kk].y & 0x7FFFu, (raw[kk].y >> 16) & 0x7FFFu)));
        }
        amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
        int kq = (int)(amax >> 7);
        kq = kq > 253 ? 253 : kq;
        const float down = pow2_of_byte(254 - kq);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            qf[kk][0] = pack_f16(__uint_as_float(raw[kk].x << 16) * down, __uint_as_float(raw[kk].x & 0xFFFF0000u) * down);
            qf[kk][1] = pack_f16(__uint_as_float(raw[kk].y << 16) * down, __uint_as_float(raw[kk].y & 0xFFFF0000u) * down);
        }
        // this thread's score columns are heads 2 tig and 2 tig + 1: their factors live in the lanes of those rows
        const float mine = p.scale_log2 * pow2_of_byte(kq);
        qmul[0] = __shfl_sync(0xffffffffu, mine, (2 * tig) * 4);
        qmul[1] = __shfl_sync(0xffffffffu, mine, (2 * tig + 1) * 4);
    }

    float o[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};                      // partial: this thread's two tokens of every block
    int eref = 0;

    const uint32_t wbase = smem_u32(smem) + warp * kWarpSmemT;
    uint64_t l2_policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(l2_policy));

#pragma unroll
    for (int s = 0; s < kStagesT - 1; ++s) {
        if (s < my_blocks) {
            const int tok0 = s0 + (warp + s * kWarps) * kBlk;
            load_block_fp8(wbase + s * kStageF8, kc, vc, ks, vs, tok0, s1, lane, l2_policy);
        }
        cp_async_commit();
    }

    for (int it = 0; it < my_blocks; ++it) {
        {
            const int nx = it + kStagesT - 1;
            if (nx < my_blocks) {
                const int tok0 = s0 + (warp + nx * kWarps) * kBlk;
                load_block_fp8(wbase + (nx % kStagesT) * kStageF8, kc, vc, ks, vs, tok0, s1, lane, l2_policy);
            }
            cp_async_commit();
        }
        cp_async_wait<kStagesT - 1>();
        __syncwarp();

        const uint32_t sk = wbase + (it % kStagesT) * kStageF8;
        const uint32_t sv = sk + kCodeBytes;
        const int tok0 = s0 + (warp + it * kWarps) * kBlk;
        const int valid = s1 - tok0;   // >= 1

        // scale bytes of this thread's two tokens, grp and grp + 8
        uint32_t kb0, kb1, vb0, vb1;
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(kb0) : "r"(sk + 2 * kCodeBytes + grp));
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(kb1) : "r"(sk + 2 * kCodeBytes + 8 + grp));
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(vb0) : "r"(sk + 2 * kCodeBytes + 16 + grp));
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(vb1) : "r"(sk + 2 * kCodeBytes + 24 + grp));
        const bool ok0 = grp < valid, ok1 = grp + 8 < valid;
        if (!ok0) { kb0 = 0; vb0 = 0; }
        if (!ok1) { kb1 = 0; vb1 = 0; }

        // S^T = K Q^T
        float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
            const int r = (lane & 7) + (((lane >> 3) & 1) << 3);
            const int c = pc * 2 + (lane >> 4);
            uint32_t m0, m1, m2, m3, a0, a1, a2, a3;
            ldmatrix_x4(sk + r * kD + ((c ^ (r & 7)) << 4), m0, m1, m2, m3);
            e4m3x4_to_f16x2x2(m0, a0, a2);      // token grp:     dims 4 tig + {0, 1} | {2, 3} of piece 2 pc
            e4m3x4_to_f16x2x2(m1, a1, a3);      // token grp + 8
            mma_f16(sc, a0, a1, a2, a3, qf[2 * pc][0], qf[2 * pc][1]);
            e4m3x4_to_f16x2x2(m2, a0, a2);      // piece 2 pc + 1
            e4m3x4_to_f16x2x2(m3, a1, a3);
            mma_f16(sc, a0, a1, a2, a3, qf[2 * pc + 1][0], qf[2 * pc + 1][1]);
        }

        // the block's largest V scale (all lanes: 16 tokens spread over the 8 row groups)
        int vmax = max((int)vb0, (int)vb1);
        vmax = max(vmax, __shfl_xor_sync(0xffffffffu, vmax, 4));
        vmax = max(vmax, __shfl_xor_sync(0xffffffffu, vmax, 8));
        vmax = max(vmax, __shfl_xor_sync(0xffffffffu, vmax, 16));
        if (vmax > eref) {
            const float f = pow2_of_byte(max(eref - vmax + 127, 0));
#pragma unroll
            for (int i = 0; i < 8; ++i) { o[i][0] *= f; o[i][1] *= f; o[i][2] *= f; o[i][3] *= f; }
            eref = vmax;
        }
        const float vf0 = pow2_of_byte(max((int)vb0 - eref + 127, 0)), vf1 = pow2_of_byte(max((int)vb1 - eref + 127, 0));
        const float kf0 = pow2_of_byte((int)kb0), kf1 = pow2_of_byte((int)kb1);

        float pr[4];                                  // probabilities: [token grp | grp + 8][head 2 tig | 2 tig + 1]
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            float t0 = ok0 ? sc[e] * (qmul[e] * kf0) : -INFINITY;
            float t1 = ok1 ? sc[2 + e] * (qmul[e] * kf1) : -INFINITY;
            float mx = fmaxf(t0, t1);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float m_new = fmaxf(m_run[e], mx);        // finite: token 0 of a block is always valid
            t0 = fast_exp2(t0 - m_new);
            t1 = fast_exp2(t1 - m_new);
            if (__any_sync(0xffffffffu, m_new > m_run[e])) {
                const float alpha = fast_exp2(m_run[e] - m_new);   // 0 on the first block
                l_run[e] = l_run[e] * alpha + (t0 + t1);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    o[i][e] *= alpha;
                    o[i][2 + e] *= alpha;
                }
            } else {
                l_run[e] += t0 + t1;
            }
            m_run[e] = m_new;
            pr[e] = t0 * vf0;
            pr[2 + e] = t1 * vf1;
        }
        // P^T for the second product: tokens along the contraction, heads along the columns
        const uint32_t pb0 = movmatrix_trans(pack_f16(pr[0], pr[1]));   // tokens 2 tig, 2 tig + 1 of head grp
        const uint32_t pb1 = movmatrix_trans(pack_f16(pr[2], pr[3]));   // tokens 8 + 2 tig, 9 + 2 tig

        // O^T += V^T P^T: a transposed 16-bit unit holds dims (2 grp, 2 grp + 1) of tokens 2 tig (low half)
        // and 2 tig + 1; the permute puts the two tokens of each dim side by side: rows grp and grp + 8 of the
        // MMA tile are dims 2 grp and 2 grp + 1 of the piece
#pragma unroll
        for (int pc = 0; pc < 4; ++pc) {
            const int r = (lane & 7) + (((lane >> 3) & 1) << 3);
            const int c = pc * 2 + (lane >> 4);
            uint32_t m0, m1, m2, m3, a0, a1, a2, a3;
            ldmatrix_x4_trans(sv + r * kD + ((c ^ (r & 7)) << 4), m0, m1, m2, m3);
            e4m3x4_to_f16x2x2(__byte_perm(m0, 0u, 0x3120), a0, a1);     // tokens 2 tig, + 1:   dim 2 grp | 2 grp + 1
            e4m3x4_to_f16x2x2(__byte_perm(m1, 0u, 0x3120), a2, a3);     // tokens 8 + 2 tig, + 1
            mma_f16(o[2 * pc], a0, a1, a2, a3, pb0, pb1);
            e4m3x4_to_f16x2x2(__byte_perm(m2, 0u, 0x3120), a0, a1);
            e4m3x4_to_f16x2x2(__byte_perm(m3, 0u, 0x3120), a2, a3);
            mma_f16(o[2 * pc + 1], a0, a1, a2, a3, pb0, pb1);
        }
        __syncwarp();
    }
    cp_async_wait<0>();
    if (p.gdc_wait) asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- stage the warp's results: rows = query heads, fp32 -------------------------------------------
    {
        const float f = pow2_of_byte(eref);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 4);
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 8);
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 16);
        }
        __syncthreads();   // every warp is done with its pipeline memory
        float* sm_o = reinterpret_cast<float*>(smem);                  // [kWarps][16][128]
        float* sm_ml = sm_o + kWarps * 16 * kD;                        // [kWarps][16][2]
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int head = 2 * tig + e;
            if (head < G) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    *reinterpret_cast<float2*>(sm_o + (warp * 16 + head) * kD + 16 * i + 2 * grp) =
                        make_float2(o[i][e] * f, o[i][2 + e] * f);
                if (grp == 0) {
                    sm_ml[(warp * 16 + head) * 2 + 0] = m_run[e];
                    sm_ml[(warp * 16 + head) * 2 + 1] = l_run[e];
                }
            }
        }
        __syncthreads();
    }
    finish_item_tail<kWarps, kD>(p, smem, &s_is_last, item, b, hg, nsplit, len_old, p.appended && p.bump_len, len_p, out_p,
                                 part_o_p, part_ml_p, counters_p, seq_counters_p);
}

template <bool HI, int kWarps>
cudaError_t setup_one_fp8() {
    return cudaFuncSetAttribute(decode_fp8_kernel<HI, kWarps>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kWarps * kWarpSmemF8);
}

}  // namespace

cudaError_t decode_fp8_setup() {
    cudaError_t e = setup_one_fp8<false, 4>();
    if (e == cudaSuccess) e = setup_one_fp8<true, 4>();
    if (e == cudaSuccess) e = setup_one_fp8<false, 8>();
    if (e == cudaSuccess) e = setup_one_fp8<true, 8>();
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(decode_fp8t_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 * kWarpSmemT);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(decode_fp8t_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * kWarpSmemT);
    return e;
}

cudaError_t launch_decode_fp8(const DecodeParams& p, int n_items, int warps, cudaStream_t s, int overlap, int n_layers) {
    if (n_items <= 0) return cudaSuccess;
    if (warps != 4 && warps != 8) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(n_items, n_layers > 0 ? n_layers : 1);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = warps * kWarpSmemF8;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    DecodeParams pp = p;
    pp.gdc_wait = (overlap == 2) ? 0 : (overlap == 3) ? 2 : 1;
    const bool hi = p.G > 8;
    cudaError_t e;
    if (!hi) {
        // groups of up to eight query heads: the transposed kernel
        cfg.dynamicSmemBytes = warps * kWarpSmemT;
        e = warps == 8 ? cudaLaunchKernelEx(&cfg, decode_fp8t_kernel<8>, pp) : cudaLaunchKernelEx(&cfg, decode_fp8t_kernel<4>, pp);
    } else if (warps == 8) {
        e = cudaLaunchKernelEx(&cfg, decode_fp8_kernel<true, 8>, pp);
    } else {
        e = cudaLaunchKernelEx(&cfg, decode_fp8_kernel<true, 4>, pp);
    }
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_quant_append(const QuantAppendParams& p, int max_new, int n_layers, cudaStream_t s) {
    const long long work = (long long)max_new * p.nR * 16;
    if (work <= 0) return cudaSuccess;
    dim3 grid((unsigned)((work + 255) / 256), p.B, n_layers > 0 ? n_layers : 1);
    quant_append_kernel<<<grid, 256, 0, s>>>(p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_dequant(const DequantParams& p, int max_len, cudaStream_t s) {
    long long blocks = ((long long)max_len * p.nR * 16 + 255) / 256;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 148 * 8) blocks = 148 * 8;
    dequant_kernel<<<dim3((unsigned)blocks, p.B), 256, 0, s>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace zz
