// Prefill attention on the 5th-generation tensor cores: tcgen05.mma with the S = Q K^T and
// O = P V accumulators in tensor memory, operands staged in shared memory by TMA.
//
// One kernel template serves both kinds of layer (compiled once per kind).  A retrieval head visits
// every KV tile up to the diagonal (causal flash attention); a streaming head visits only the tiles that can hold
// visible keys -- the sink tiles and the local band -- and applies the token-exact
// visibility rule inside them (block sparsity is an execution strategy, not the mask).
// Keys come from two places: the store as it stood before the call (append-only rows, contiguous
// or in 128-token pages; or ring slots, whose tokens follow from the length) and the new chunk.
//
// Work item = one 128-token query tile x two query heads of the same KV head, so each K/V tile is
// fetched once for two score tiles and the two tiles ping-pong on the tensor pipe.  A CTA works
// through a static share of the items (one CTA per SM; one item per CTA when a launch has no more
// items than SMs):
//   warps 0-3   softmax / correction / epilogue of tile 0 (one thread per query row)
//   warps 4-7   the same for tile 1
//   warp 8      TMA producer (one elected lane)
//   warp 9      MMA issuer   (one elected lane)
//   warps 10-11 idle: they only complete the third warpgroup, which hands most of its registers
//               to the two softmax warpgroups (setmaxnreg)
// Tensor memory (512 columns): tile t has S_t at column 256 t (128 fp32 columns; the bf16
// probabilities P_t overwrite its first 64 columns and feed the PV MMA as the A operand from
// tensor memory) and O_t at column 256 t + 128.
// Every mbarrier wait is bounded; when one expires the kernel records ZZ_ERR_TIMEOUT in the
// status word, stops waiting long for anything else, frees its tensor memory and returns.
#include <cuda.h>

#include "zz_common.cuh"

namespace zz {

namespace {

constexpr int kTile = 128;
constexpr int kSubBytes = 128 * 128;        // [128 rows][64 bf16] sub-tile, 128-byte swizzled
constexpr int kTileBytes = 2 * kSubBytes;   // a full [128][128] bf16 tile (head_dim 128; half of it at head_dim 64)
constexpr int kStages = 4;                  // K/V tiles held at once: two pair slots of (V_j, K_{j+1})
constexpr int kPairs = 2;                   // one full / empty barrier per pair: what an iteration uses, it uses together
constexpr int kThreads = 384;                // three warpgroups: softmax tile 0, softmax tile 1, TMA + MMA
constexpr int kWarpTma = 8, kWarpMma = 9;
constexpr int kRegsSoftmax = 200, kRegsAux = 104;  // 200 * 256 + 104 * 128 = 64512 registers, what the launch allocates (168 * 384)
constexpr int kEpiBytes = 8 * 4096;          // output staging: 16 rows of 256 B per softmax warp
constexpr int kMaxOrder = 768;               // items of one CTA that can be re-ordered (2 bytes each)
constexpr int kMaxOrderKeys = 1024;          // distinct (sequence, KV head) keys the re-ordering handles
constexpr int kOrderBytes = kMaxOrder * 2;
constexpr int kSmemBytes = 2 * kTileBytes + kStages * kTileBytes + kEpiBytes + kOrderBytes + 1024;
constexpr uint32_t kMaxPolls = 1u << 22;
constexpr uint32_t kAbortPolls = 1u << 10;
constexpr float kRescaleThreshold = 8.f;    // log2 units of slack before O is rescaled
#ifndef ZZ_POLY_EVERY
#define ZZ_POLY_EVERY 8
#endif
constexpr int kPolyEvery = ZZ_POLY_EVERY;   // one pair in kPolyEvery takes the polynomial exp2 (>= 17: none)

// instruction descriptor: fp32 accumulate, bf16 A and B, M = 128, N = 128
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
// P V: N = head_dim, B (= V) is MN-major
__host__ __device__ constexpr uint32_t idesc_pv(int hd) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (((uint32_t)hd >> 3) << 17) | ((128u >> 4) << 24);
}

struct Shared {
    uint64_t q_full;
    uint64_t q_empty;          // the item's last Q K^T has completed: the Q buffer may be reloaded
    uint64_t kv_full[kPairs];
    uint64_t kv_empty[kPairs];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t o_full[2];        // per query tile: its last P V has completed
    uint32_t tmem_base;
    uint32_t poll_limit;       // probes a wait may spend before it gives up (kMaxPolls in the product kernels)
    int abort_flag;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (after flagging the error) if the phase never completed.
// The first probe is inlined: a wait on a phase that has already completed costs one
// try_wait, and only a real wait enters the polling loop.
__device__ __forceinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, Shared* sh, int* status) {
    const uint32_t limit = (*(volatile int*)&sh->abort_flag) ? (uint32_t)kAbortPolls : (uint32_t)(*(volatile uint32_t*)&sh->poll_limit);
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 4095u) == 4095u && (*(volatile int*)&sh->abort_flag)) break;
    }
    *(volatile int*)&sh->abort_flag = 1;
    atomicExch(status, ZZ_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Shared* sh, int* status) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, sh, status);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}

// shared-memory matrix descriptor, 128-byte swizzle, sm_100 descriptor version
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}

// Descriptors travel as (low word, high word): only the low word (start address >> 4 in its 14
// low bits) changes between the MMAs of a tile, so stepping one costs a single 32-bit add.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t ab_hi_a,
                                       uint32_t ab_hi_b, uint32_t idesc, bool acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(ab_hi_a), "r"(b_lo), "r"(ab_hi_b), "r"(idesc), "r"((uint32_t)acc)
        : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                       uint32_t idesc, bool acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"((uint32_t)acc)
        : "memory");
}
// Predicated forms (exec == 0: the instruction is issued but has no effect).  The thread that
// issues the MMAs must not branch between them: the tensor pipe holds next to no queue, so every
// cycle that thread spends resolving a branch is a cycle the pipe idles.
__device__ __forceinline__ void mma_ss_if(uint32_t exec, uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_hi,
                                          uint32_t b_hi, uint32_t idesc, bool acc) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\tsetp.ne.b32 q, %7, 0;\n\t"
        "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"((uint32_t)acc), "r"(exec)
        : "memory");
}
__device__ __forceinline__ void mma_commit_if(uint32_t exec, uint64_t* bar) {
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(smem_u32(bar)), "r"(exec)
        : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets lane (base + i)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
// 32 lanes x 128 consecutive fp32 columns in one instruction
__device__ __forceinline__ void tmem_ld128(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x128.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63,%64,%65,%66,%67,%68,%69,%70,%71,%72,%73,%74,%75,%76,%77,%78,%79,%80,%81,%82,%83,%84,%85,%86,%87,%88,%89,%90,%91,%92,%93,%94,%95,%96,%97,%98,%99,%100,%101,%102,%103,%104,%105,%106,%107,%108,%109,%110,%111,%112,%113,%114,%115,%116,%117,%118,%119,%120,%121,%122,%123,%124,%125,%126,%127}, [%128];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63]), "=r"(r[64]), "=r"(r[65]), "=r"(r[66]), "=r"(r[67]), "=r"(r[68]), "=r"(r[69]), "=r"(r[70]), "=r"(r[71]), "=r"(r[72]), "=r"(r[73]), "=r"(r[74]), "=r"(r[75]), "=r"(r[76]), "=r"(r[77]), "=r"(r[78]), "=r"(r[79]), "=r"(r[80]), "=r"(r[81]), "=r"(r[82]), "=r"(r[83]), "=r"(r[84]), "=r"(r[85]), "=r"(r[86]), "=r"(r[87]), "=r"(r[88]), "=r"(r[89]), "=r"(r[90]), "=r"(r[91]), "=r"(r[92]), "=r"(r[93]), "=r"(r[94]), "=r"(r[95]), "=r"(r[96]), "=r"(r[97]), "=r"(r[98]), "=r"(r[99]), "=r"(r[100]), "=r"(r[101]), "=r"(r[102]), "=r"(r[103]), "=r"(r[104]), "=r"(r[105]), "=r"(r[106]), "=r"(r[107]), "=r"(r[108]), "=r"(r[109]), "=r"(r[110]), "=r"(r[111]), "=r"(r[112]), "=r"(r[113]), "=r"(r[114]), "=r"(r[115]), "=r"(r[116]), "=r"(r[117]), "=r"(r[118]), "=r"(r[119]), "=r"(r[120]), "=r"(r[121]), "=r"(r[122]), "=r"(r[123]), "=r"(r[124]), "=r"(r[125]), "=r"(r[126]), "=r"(r[127])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
    const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
          "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// two fp32 lanes per instruction (packed FMA / ADD of sm_100)
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "mov.b64 rc, {%6, %7};\n\tfma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 add2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
// 2^x for a pair of x <= ~120 on the FMA pipe instead of the MUFU: x = n + f with n = round(x)
// (taken from the low mantissa bits of x + 1.5 * 2^23) and f in [-0.5, 0.5]; 2^f by a cubic
// fitted to minimise the relative error on that interval (7.5e-5, far below the bf16 rounding of
// the probabilities); n goes straight into the exponent field.
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
    const float kMagic = 12582912.f;
    // below 2^-126 the exponent arithmetic at the end would wrap around; such probabilities are zero
    // to the row sum and to the bf16 operand alike, so the argument is held at -126
    x.x = fmaxf(x.x, -126.f);
    x.y = fmaxf(x.y, -126.f);
    const float2 t = add2(x, make_float2(kMagic, kMagic));
    const float2 r = add2(t, make_float2(-kMagic, -kMagic));
    const float2 f = fma2(r, make_float2(-1.f, -1.f), x);
    float2 p = fma2(make_float2(0.055171408f, 0.055171408f), f, make_float2(0.24261075f, 0.24261075f));
    p = fma2(p, f, make_float2(0.69326097f, 0.69326097f));
    p = fma2(p, f, make_float2(0.99992812f, 0.99992812f));
    float2 o;
    o.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
    o.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
    return o;
}

// bits i of a 32-bit word that stand for columns base + i inside [lo, hi]
__device__ __forceinline__ uint32_t range_bits(int lo, int hi, int base) {
    const int a = max(lo - base, 0), b = min(hi - base, 31);
    if (a > b) return 0u;
    return (0xffffffffu >> (31 - b)) & (0xffffffffu << a);
}

// Which KV tiles a query tile visits, in order: store tiles, then chunk tiles (sink tiles of
// the chunk that lie before the band, then the band up to the diagonal).
struct TilePlan {
    int n_store;       // tiles over the store (rows 0.. of the append-only store / ring slots)
    int n_sink_chunk;  // leading chunk tiles visited only for their sinks
    int band_lo;       // first chunk tile of the band
    int n_total;
    int n_occ;         // occupied store rows (P, or min(P, S+W))
};

__device__ __forceinline__ TilePlan make_plan(int kind, int P, int C, int qt, int S, int W, int ring) {
    TilePlan t;
    const int r0 = qt * kTile;
    if (kind == ZZ_KIND_RETRIEVAL) {
        t.n_occ = P;
        t.n_store = (P + kTile - 1) / kTile;
        t.n_sink_chunk = 0;
        t.band_lo = 0;
    } else {
        t.n_occ = min(P, ring);
        const int full = (t.n_occ + kTile - 1) / kTile;
        const int sink_tiles = (min(S, t.n_occ) + kTile - 1) / kTile;
        t.n_store = (r0 < W) ? full : sink_tiles;   // rows >= W see no recent key of the old store
        const int n_sink_c = max(0, min(S - P, C));
        const int ns = (n_sink_c + kTile - 1) / kTile;
        const int lo = r0 - W + 1;
        t.band_lo = lo > 0 ? lo / kTile : 0;
        t.n_sink_chunk = min(ns, t.band_lo);
    }
    t.n_total = t.n_store + t.n_sink_chunk + (qt - t.band_lo + 1);
    return t;
}

// tile j of the plan: from the store (is_chunk = false) or the chunk, starting at row `start`
__device__ __forceinline__ void plan_tile(const TilePlan& t, int j, bool& is_chunk, int& start) {
    if (j < t.n_store) {
        is_chunk = false;
        start = j * kTile;
    } else {
        is_chunk = true;
        const int c = j - t.n_store;
        start = (c < t.n_sink_chunk ? c : t.band_lo + (c - t.n_sink_chunk)) * kTile;
    }
}

// One work item = (128-token query tile, KV head of the group, pair of query heads).  A CTA is
// persistent: it works through items k = 0, 1, ... of a static boustrophedon schedule over the
// items in long-first order (wave w forwards, wave w+1 backwards), so every CTA gets nearly the same
// number of KV tiles, the TMA producer runs ahead into the next item, and tensor-memory allocation,
// barrier set-up and the first loads are paid once per CTA instead of once per item.
struct Item {
    int b, qt, r0, C, P, hg, g0, n_tiles;
    bool active1;
    TilePlan plan;
};
__device__ __forceinline__ int item_index(int k, int n_items) {
    const int g = (int)gridDim.x;
    const int idx = k * g + ((k & 1) ? g - 1 - (int)blockIdx.x : (int)blockIdx.x);
    return idx < n_items ? idx : -1;
}
__device__ __forceinline__ Item get_item(const PrefillParams& p, int kind, int idx) {
    Item it;
    const int pairs = (p.G + 1) >> 1;
    const int per_tile = p.Hg * pairs;
    const int ti = idx / per_tile;
    const int rem = idx % per_tile;
    it.hg = rem / pairs;
    it.g0 = (rem % pairs) * 2;
    it.active1 = (it.g0 + 1) < p.G;
    const int gt = p.total_tiles - 1 - ti;      // long (late) tiles first
    int b = 0;
    while (b + 1 < p.B && gt >= p.tile_start[b + 1]) ++b;
    it.b = b;
    it.qt = gt - p.tile_start[b];
    it.r0 = it.qt * kTile;
    it.C = p.n_new[b];
    it.P = p.len[b];
    it.plan = make_plan(kind, it.P, it.C, it.qt, p.S, p.W, p.ring);
    it.n_tiles = it.plan.n_total;
    return it;
}
// (sequence, KV head) of an item as one number: items with equal keys read the same K/V rows
__device__ __forceinline__ int item_key(const PrefillParams& p, int idx) {
    const int pairs = (p.G + 1) >> 1;
    const int per_tile = p.Hg * pairs;
    const int gt = p.total_tiles - 1 - idx / per_tile;
    int b = 0;
    while (b + 1 < p.B && gt >= p.tile_start[b + 1]) ++b;
    return b * p.Hg + (idx % per_tile) / pairs;
}

// kPersistent = false: one item per CTA (grid = items, for launches with no more items than SMs);
// the item loops below then run once and every running counter folds to a constant.  Persistent
// CTAs gain ~10 % on the short items of streaming layers and 2-5 % on retrieval chunks of 2K-8K
// tokens; on 32K chunks the two time the same.
// HD = head_dim: 128, or 64 (Q, K and V tiles are then one 64-column sub-tile, Q K^T has four MMA steps
// instead of eight, P V has N = 64, and O takes 64 columns of tensor memory).
// kStreaming: the kind of layer (compiled apart: a retrieval launch carries none of the ring and window
// arithmetic, and the short items of a streaming launch end each query tile on a barrier of its own).
template <bool kPersistent, int HD, bool kStreaming>
__global__ void __launch_bounds__(kThreads, 1)
prefill_kernel(const PrefillParams p, const __grid_constant__ CUtensorMap tmap_q,
               const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
               const __grid_constant__ CUtensorMap tmap_arena) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ Shared sh;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sm_q = smem_base;                       // two Q tiles
    constexpr int kTileB = (HD / 64) * kSubBytes;          // bytes of a Q, K or V tile
    constexpr uint32_t kIdescPV = idesc_pv(HD);
    const uint32_t sm_kv = smem_base + 2 * kTileBytes;     // kStages K/V tiles

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kind = kStreaming ? ZZ_KIND_STREAMING : ZZ_KIND_RETRIEVAL;

    const int n_items = p.n_items;
    const uint32_t sm_epi = smem_base + 2 * kTileBytes + kStages * kTileBytes;   // output staging

    // ---- this CTA's items and the order it takes them in ------------------------------------------
    // The static schedule hands CTA c the items k * grid + snake(c), k = 0 .. n_mine - 1, of the
    // long-first numbering (equal work per CTA).  A retrieval launch walks its share sorted by
    // (sequence, KV head) instead: all CTAs then stream the same one or two KV heads at any time, whose
    // K/V rows fit the L2, instead of all heads at once (K/V came from HBM 4-11 times over).  The sort
    // is stable, so within a head the long items still come first.
    int n_mine = 1;
    bool use_order = false;
    if (kPersistent) {
        const int g = (int)gridDim.x, full = n_items / g, rem = n_items % g;
        const int pos = (full & 1) ? g - 1 - (int)blockIdx.x : (int)blockIdx.x;
        n_mine = full + (pos < rem ? 1 : 0);
        use_order = kind == ZZ_KIND_RETRIEVAL && n_mine > 2 && n_mine <= kMaxOrder && p.B * p.Hg <= kMaxOrderKeys &&
                    p.B * p.Hg > 1;
    }
    unsigned char* const smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    uint16_t* const sm_order = reinterpret_cast<uint16_t*>(smem_gen + 2 * kTileBytes + kStages * kTileBytes + kEpiBytes);
    if (kPersistent && use_order && warp == 10) {
        uint16_t* const cnt = reinterpret_cast<uint16_t*>(smem_gen + 2 * kTileBytes + kStages * kTileBytes);  // scratch: the staging area
        const int nkeys = p.B * p.Hg;
        for (int i = lane; i < nkeys; i += 32) cnt[i] = 0;
        __syncwarp();
        for (int k0 = 0; k0 < n_mine; k0 += 32) {          // how many of my items each key has
            const int k = k0 + lane;
            const bool valid = k < n_mine;
            const int key = valid ? item_key(p, item_index(k, n_items)) : -1 - lane;
            const unsigned m = __match_any_sync(0xffffffffu, key);
            if (valid && lane == __ffs(m) - 1) cnt[key] += (uint16_t)__popc(m);
            __syncwarp();
        }
        int carry = 0;
        for (int i0 = 0; i0 < nkeys; i0 += 32) {             // exclusive prefix sum: first position of each key
            const int i = i0 + lane;
            const int v = i < nkeys ? cnt[i] : 0;
            int incl = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            if (i < nkeys) cnt[i] = (uint16_t)(carry + incl - v);
            carry += __shfl_sync(0xffffffffu, incl, 31);
            __syncwarp();
        }
        for (int k0 = 0; k0 < n_mine; k0 += 32) {          // stable scatter
            const int k = k0 + lane;
            const bool valid = k < n_mine;
            const int key = valid ? item_key(p, item_index(k, n_items)) : -1 - lane;
            const unsigned m = __match_any_sync(0xffffffffu, key);
            if (valid) sm_order[cnt[key] + __popc(m & ((1u << lane) - 1u))] = (uint16_t)k;
            __syncwarp();
            if (valid && lane == __ffs(m) - 1) cnt[key] += (uint16_t)__popc(m);
            __syncwarp();
        }
    }
    // item k of this CTA (or -1 past the last one)
    auto my_item = [&](int k) -> int {
        if (!kPersistent) return (int)blockIdx.x;
        if (k >= n_mine) return -1;
        return item_index(use_order ? (int)sm_order[k] : k, n_items);
    };

    if (threadIdx.x == 0) {
        mbar_init(&sh.q_full, 1);
        mbar_init(&sh.q_empty, 1);
        for (int i = 0; i < kPairs; ++i) {
            mbar_init(&sh.kv_full[i], 1);
            mbar_init(&sh.kv_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh.s_full[i], 1);
            mbar_init(&sh.p_full[i], 128);
        }
        mbar_init(&sh.o_full[0], 1);
        mbar_init(&sh.o_full[1], 1);
        sh.poll_limit = kMaxPolls;
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kWarpTma) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sh.tmem_base))
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *(volatile uint32_t*)&sh.tmem_base;

    // Registers move from the TMA/MMA warpgroup (which needs few) to the softmax warpgroups, whose
    // threads each hold a 128-column row of scores.
    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsAux));
      if (warp == kWarpTma) {
        // ================= TMA producer =================
        if (lane == 0) {
            uint32_t u_glob = 0;                      // K/V pairs loaded so far (all items)
            for (int k = 0;; ++k) {
                if (!kPersistent && k > 0) break;
                const int idx = my_item(k);
                if (idx < 0) break;
                const Item it = get_item(p, kind, idx);
                const SeqDesc sd = p.desc[it.b];
                const long long slots_per_head = (kind == ZZ_KIND_RETRIEVAL) ? sd.cap : p.ring;
                // paged retrieval store: a store tile is one page (tiles and pages are both 128 tokens)
                const bool paged = p.page_table != nullptr && kind == ZZ_KIND_RETRIEVAL;
                const int* const tbl = paged ? p.page_table + sd.tbl + it.hg : nullptr;
                const int k_row0 = (int)(sd.k_off[kind] / HD + (paged ? 0ll : (long long)it.hg * slots_per_head));
                const int v_row0 = (int)(sd.v_off[kind] / HD + (paged ? 0ll : (long long)it.hg * slots_per_head));
                const int src_head = p.head_list[p.kv_head0 + it.hg];
                const int tok0 = p.tok_off[it.b];
                const int qh = p.q_head0 + it.hg * p.G + it.g0;
                if (k > 0) mbar_wait(&sh.q_empty, (k - 1) & 1, &sh, p.status);
                mbar_expect_tx(&sh.q_full, it.active1 ? 2 * kTileB : kTileB);
                tma_load_3d(sm_q, &tmap_q, 0, qh, tok0 + it.r0, &sh.q_full);
                if (HD == 128) tma_load_3d(sm_q + kSubBytes, &tmap_q, 64, qh, tok0 + it.r0, &sh.q_full);
                if (it.active1) {
                    tma_load_3d(sm_q + kTileB, &tmap_q, 0, qh + 1, tok0 + it.r0, &sh.q_full);
                    if (HD == 128) tma_load_3d(sm_q + kTileB + kSubBytes, &tmap_q, 64, qh + 1, tok0 + it.r0, &sh.q_full);
                }
                // pair pi of the item: pi = 0 holds K_0 alone, pi = j + 1 holds (V_j, K_{j+1}), the last one
                // V_{n-1} alone; slot = running pair count % 2, V in the slot's first tile, K in its second
                for (int pi = 0; pi <= it.n_tiles; ++pi, ++u_glob) {
                    const int slot = u_glob % kPairs;
                    mbar_wait(&sh.kv_empty[slot], ((u_glob / kPairs) & 1) ^ 1, &sh, p.status);
                    const bool has_v = pi > 0, has_k = pi < it.n_tiles;
                    mbar_expect_tx(&sh.kv_full[slot], (has_v && has_k) ? 2 * kTileB : kTileB);
#pragma unroll
                    for (int is_k = 0; is_k < 2; ++is_k) {
                        if (is_k ? !has_k : !has_v) continue;
                        bool is_chunk;
                        int start;
                        plan_tile(it.plan, is_k ? pi : pi - 1, is_chunk, start);
                        const uint32_t dst = sm_kv + (slot * 2 + is_k) * kTileB;
                        if (is_chunk) {
                            const CUtensorMap* m = is_k ? &tmap_k : &tmap_v;
                            tma_load_3d(dst, m, 0, src_head, tok0 + start, &sh.kv_full[slot]);
                            if (HD == 128) tma_load_3d(dst + kSubBytes, m, 64, src_head, tok0 + start, &sh.kv_full[slot]);
                        } else {
                            const int row = (is_k ? k_row0 : v_row0) +
                                            (paged ? tbl[(start >> 7) * p.Hg] * (int)(kPageElems / kD) : start);
                            tma_load_2d(dst, &tmap_arena, 0, row, &sh.kv_full[slot]);
                            if (HD == 128) tma_load_2d(dst + kSubBytes, &tmap_arena, 64, row, &sh.kv_full[slot]);
                        }
                    }
                }
            }
        }
      } else if (warp == kWarpMma) {
        // ================= MMA issuer =================
        // The whole warp runs this loop and its barrier waits; one lane issues the MMAs and commits.
        // Measured on this hardware: an issuing thread that sits alone in a divergent branch is
        // starved of issue slots by the softmax warps of its SM sub-partition (a tile's 16 MMAs took
        // up to 3x their 1024 cycles next to a busy warp), a warp in uniform control flow is not
        // (1.1x).  Everything the descriptors derive from is made provably warp-uniform for the
        // same reason.
        {
            const bool leader = lane == 0;
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
            const uint64_t dq = make_desc(sm_q, 16, 1024);          // Q tile 0, K-major
            const uint64_t dk = make_desc(sm_kv, 16, 1024);         // K tile of pair slot 0, K-major
            const uint64_t dv = make_desc(sm_kv, kSubBytes, 1024);  // V tile of pair slot 0, MN-major
            const uint32_t dq_lo = (uint32_t)dq, dk_lo = (uint32_t)dk, dv_lo = (uint32_t)dv;
            const uint32_t dkm_hi = (uint32_t)(dq >> 32), dv_hi = (uint32_t)(dv >> 32);
            constexpr uint32_t kTile16 = kTileB >> 4;
            // Counters that run across the items of this CTA (barrier phases never restart):
            uint32_t u_glob = 0;          // K/V pairs consumed
            uint32_t ph[2] = {0, 0};      // S/P tiles handled per query tile (tile 1 only in items that have it)
            for (int k = 0;; ++k) {
                if (!kPersistent && k > 0) break;
                const int idx = my_item(k);
                if (idx < 0) break;
                const Item it = get_item(p, kind, idx);
                const int n_tiles = __shfl_sync(0xffffffffu, it.n_tiles, 0);
                const bool active1 = it.active1;
                const int n_act = active1 ? 2 : 1;
                mbar_wait(&sh.q_full, k & 1, &sh, p.status);
                mbar_wait(&sh.kv_full[u_glob % kPairs], (u_glob / kPairs) & 1, &sh, p.status);
                tc_fence_after();
                if (leader) {
                    // S_t = Q_t K_0^T
                    for (int t = 0; t < n_act; ++t) {
#pragma unroll
                        for (int kk = 0; kk < HD / 16; ++kk) {
                            const uint32_t off16 = (kk >> 2) * (kSubBytes >> 4) + (kk & 3) * 2;
                            mma_ss(tmem_u + t * 256, dq_lo + t * kTile16 + off16,
                                   dk_lo + ((u_glob % kPairs) * 2 + 1) * kTile16 + off16, dkm_hi, dkm_hi, kIdescQK, kk > 0);
                        }
                        mma_commit(&sh.s_full[t]);
                    }
                    mma_commit(&sh.kv_empty[u_glob % kPairs]);
                    if (kPersistent) mma_commit_if(n_tiles == 1, &sh.q_empty);
                }
                __syncwarp();
                for (int j = 0; j < n_tiles; ++j) {
                    const uint32_t pj = u_glob + 1 + j;             // the pair (V_j, K_{j+1})
                    const uint32_t slot = pj % kPairs;
                    const uint32_t more = (j + 1) < n_tiles;
                    const uint32_t dvj = dv_lo + (slot * 2) * kTile16, dkj = dk_lo + (slot * 2 + 1) * kTile16;
                    mbar_wait(&sh.kv_full[slot], (pj / kPairs) & 1, &sh, p.status);
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (t == 1 && !active1) break;
                        mbar_wait(&sh.p_full[t], (ph[t] + j) & 1, &sh, p.status);
                        tc_fence_after();
                        if (leader) {
                            const uint32_t t_st = tmem_u + t * 256;
                            const uint32_t dqt = dq_lo + t * kTile16;
                            const uint32_t last_of_iter = (t == 1) ? 1u : (active1 ? 0u : 1u);
                            // O_t (+)= P_t V_j
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk)
                                mma_ts(t_st + 128, t_st + kk * 8, dvj + kk * (2048 >> 4), dv_hi, kIdescPV,
                                       (kk > 0) || (j > 0));
                            // S_t = Q_t K_{j+1}^T (not after the last tile)
#pragma unroll
                            for (int kk = 0; kk < HD / 16; ++kk) {
                                const uint32_t off16 = (kk >> 2) * (kSubBytes >> 4) + (kk & 3) * 2;
                                mma_ss_if(more, t_st, dqt + off16, dkj + off16, dkm_hi, dkm_hi, kIdescQK, kk > 0);
                            }
                            // Commits cost tensor-pipe time beyond the first one after an MMA group, so
                            // there is one per tile (its S) plus one per iteration (the K/V pair is free)
                            mma_commit_if(more, &sh.s_full[t]);
                            // the tile's last P V: its O is final (in a streaming launch each query tile has
                            // its own barrier, so the epilogue of one does not wait for the other's last
                            // softmax; in a retrieval launch, whose items are long, one commit per item after
                            // the loop keeps this instruction stream as short as it can be)
                            if constexpr (kStreaming) mma_commit_if(more ^ 1u, &sh.o_full[t]);
                            mma_commit_if(last_of_iter, &sh.kv_empty[slot]);
                            // after the item's last Q K^T the Q buffer may take the next item's tiles
                            if (kPersistent) mma_commit_if((j + 2 == n_tiles) & last_of_iter, &sh.q_empty);
                        }
                        __syncwarp();
                    }
                }
                if constexpr (!kStreaming) {
                    if (leader) mma_commit(&sh.o_full[0]);
                    __syncwarp();
                }
                u_glob += n_tiles + 1;
                ph[0] += n_tiles;
                if (active1) ph[1] += n_tiles;
            }
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        // ================= softmax / correction / epilogue =================
        const int t = warp >> 2;                        // which of the two tiles
        const int quarter = warp & 3;                   // tensor-memory lanes this warp may touch
        const uint32_t t_s = tmem + ((uint32_t)(quarter * 32) << 16) + t * 256;
        const uint32_t t_o = t_s + 128;
        const float sc = p.scale_log2;
        uint32_t ph = 0;                                // S/P tiles of this query tile handled so far
        uint32_t n_done = 0;                            // items this warpgroup has finished
        for (int k = 0;; ++k) {
            if (!kPersistent && k > 0) break;
            const int item_idx = my_item(k);
            if (item_idx < 0) break;
            const Item it = get_item(p, kind, item_idx);
            if (t == 1 && !it.active1) continue;
            const int n_tiles = it.n_tiles, r0 = it.r0, C = it.C, P = it.P, b = it.b, hg = it.hg, g0 = it.g0;
            const TilePlan plan = it.plan;
            const int r = quarter * 32 + lane;          // query row inside the tile
            const int rr = r0 + r;                      // row inside the chunk
            float m_used = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n_tiles; ++j) {
                bool is_chunk;
                int start;
                plan_tile(plan, j, is_chunk, start);
                // ---- visibility (decided while S is still being computed: measured 1.6 % on an 8K chunk) ----
                // tile_masked: some entry of this 128 x 128 tile may be invisible (uniform over the
                // CTA); vis[w] bit i: column 32 w + i is visible to this thread's row
                bool tile_masked = true;
                if (kind == ZZ_KIND_RETRIEVAL) {
                    tile_masked = is_chunk ? (start + 127 > r0) : (plan.n_occ - start < 128);
                } else if (is_chunk) {
                    // a chunk tile of a streaming layer is fully visible to all 128 rows if it lies
                    // below the diagonal and either inside every row's window or among the sinks
                    const bool below = start + 127 <= r0;
                    const bool in_window = start >= r0 + 127 - p.W + 1;
                    const bool all_sinks = start + 127 < p.S - P;
                    tile_masked = !(below && (in_window || all_sinks));
                }
                mbar_wait(&sh.s_full[t], (ph + j) & 1, &sh, p.status);
                tc_fence_after();
                float s[128];
                tmem_ld128(t_s, s);
                tmem_wait_ld();
                if (tile_masked) {
                    uint32_t vis[4];
                    if (kind == ZZ_KIND_RETRIEVAL) {
                        // store rows past the store's length; causal inside the chunk
                        const int lim = is_chunk ? (rr - start + 1) : (plan.n_occ - start);
#pragma unroll
                        for (int w = 0; w < 4; ++w) vis[w] = range_bits(0, lim - 1, 32 * w);
                    } else if (!is_chunk) {
                        // Ring slots visible to the query at position tq: the sinks, and the stored tokens
                        // t >= tq - W + 1.  After P appended tokens the ring holds tokens max(S, P - W) .. P - 1
                        // at slots S + ((t - S) mod W), so a run of consecutive tokens is a run of consecutive
                        // slots that wraps at most once: three slot ranges instead of a look-up per column.
                        const int tq = P + rr;
                        const int n_sink = min(p.S, P);
                        const int lo_t = max(max(p.S, P - p.W), tq - p.W + 1);   // first visible stored non-sink token
                        const int n_rec = max(P - lo_t, 0);
                        const int a = p.S + (lo_t - p.S) % p.W;                  // its slot
                        const int e1 = min(a + n_rec, p.ring);                   // end of the run before the wrap
                        const int wrap = a + n_rec - e1;                         // slots of the run after the wrap
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            const int base = start + 32 * w;
                            vis[w] = range_bits(0, n_sink - 1, base) |
                                     (n_rec > 0 ? range_bits(a, e1 - 1, base) | range_bits(p.S, p.S + wrap - 1, base) : 0u);
                        }
                    } else {
                        const int c_hi = rr - start;                      // causal
                        const int c_lo = rr - p.W + 1 - start;            // window
                        const int c_sink = p.S - P - start;               // chunk tokens that are sinks
#pragma unroll
                        for (int w = 0; w < 4; ++w)
                            vis[w] = range_bits(0, c_hi, 32 * w) &
                                     (range_bits(c_lo, 127, 32 * w) | range_bits(0, c_sink - 1, 32 * w));
                    }
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if (!((vis[c >> 5] >> (c & 31)) & 1u)) s[c] = -INFINITY;
                }

                // ---- probabilities p = 2^(s * scale - m) as bf16 into tensor memory, fp32 row sum ----
                // m is any upper estimate of the row maximum that keeps 2^(s * scale - m) finite, so the
                // exponentials do not wait for this tile's maximum: they are taken against the running
                // m, the tile's maximum is reduced alongside them (other pipe, no dependency), and only if
                // it exceeds m by more than the threshold is m raised, O rescaled and the tile redone.
                // The MUFU evaluates 16 exponentials per clock and SM, which for a 128 x 128 tile is as
                // long as its two MMAs; on tiles without masked (-inf) entries every kPolyEvery-th
                // pair is therefore evaluated by a polynomial on the FMA pipe instead.
                float psum = 0.f;
                // The common tile (nothing masked, not the item's first) runs straight through: every
                // uniform branch between "S is here" and "P is there" costs tens of cycles on the path
                // that the tensor pipe waits for.  If the maximum did move, the general loop below redoes it.
                bool done = false;
                if (!tile_masked && j > 0) {
                    // (a row that has seen nothing yet has m_used = -inf: any finite score then counts as a
                    // move of the maximum, and the general loop takes over)
                    const float msub = (m_used == -INFINITY) ? 0.f : m_used;
                    const float2 sc2 = make_float2(sc, sc), nm2 = make_float2(-msub, -msub);
                    float2 ps2 = make_float2(0.f, 0.f);
                    float mc[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t pk[16];
                        float a = s[c * 32];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const float s0 = s[c * 32 + 2 * i], s1 = s[c * 32 + 2 * i + 1];
                            a = max3(a, s0, s1);
                            const float2 x = fma2(make_float2(s0, s1), sc2, nm2);
                            const float2 e = ((i % kPolyEvery) == kPolyEvery - 1)
                                                 ? exp2_poly2(x)
                                                 : make_float2(fast_exp2(x.x), fast_exp2(x.y));
                            ps2 = add2(ps2, e);
                            pk[i] = pack_bf16(e.x, e.y);
                        }
                        mc[c] = a;
                        tmem_st16(t_s + c * 16, pk);
                    }
                    const float mx = fmaxf(max3(mc[0], mc[1], mc[2]), mc[3]) * sc;
                    if (!__any_sync(0xffffffffu, mx > m_used + kRescaleThreshold)) {
                        psum = ps2.x + ps2.y;
                        done = true;
                    }
                }
#pragma unroll 1
                for (int attempt = done ? 2 : 0; attempt < 2; ++attempt) {
                    const bool do_exp = (attempt == 1) || (j > 0);
                    float mc[4];
                    if (do_exp) {
                        const float msub = (m_used == -INFINITY) ? 0.f : m_used;
                        const float2 sc2 = make_float2(sc, sc), nm2 = make_float2(-msub, -msub);
                        float2 ps2 = make_float2(0.f, 0.f);
                        if (tile_masked) {
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                uint32_t pk[16];
                                float a = s[c * 32];
#pragma unroll
                                for (int i = 0; i < 16; ++i) {
                                    const float s0 = s[c * 32 + 2 * i], s1 = s[c * 32 + 2 * i + 1];
                                    a = max3(a, s0, s1);
                                    const float2 x = fma2(make_float2(s0, s1), sc2, nm2);
                                    const float2 e = make_float2(fast_exp2(x.x), fast_exp2(x.y));
                                    ps2 = add2(ps2, e);
                                    pk[i] = pack_bf16(e.x, e.y);
                                }
                                mc[c] = a;
                                tmem_st16(t_s + c * 16, pk);
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                uint32_t pk[16];
                                float a = s[c * 32];
#pragma unroll
                                for (int i = 0; i < 16; ++i) {
                                    const float s0 = s[c * 32 + 2 * i], s1 = s[c * 32 + 2 * i + 1];
                                    a = max3(a, s0, s1);
                                    const float2 x = fma2(make_float2(s0, s1), sc2, nm2);
                                    const float2 e = ((i % kPolyEvery) == kPolyEvery - 1)
                                                         ? exp2_poly2(x)
                                                         : make_float2(fast_exp2(x.x), fast_exp2(x.y));
                                    ps2 = add2(ps2, e);
                                    pk[i] = pack_bf16(e.x, e.y);
                                }
                                mc[c] = a;
                                tmem_st16(t_s + c * 16, pk);
                            }
                        }
                        psum = ps2.x + ps2.y;
                    } else {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            float a = s[c * 32];
#pragma unroll
                            for (int i = 0; i < 16; ++i) a = max3(a, s[c * 32 + 2 * i], s[c * 32 + 2 * i + 1]);
                            mc[c] = a;
                        }
                    }
                    if (attempt == 1) break;
                    const float mx = fmaxf(max3(mc[0], mc[1], mc[2]), mc[3]) * sc;
                    const bool bump = mx > m_used + kRescaleThreshold || (m_used == -INFINITY && mx > -INFINITY);
                    if (do_exp && !__any_sync(0xffffffffu, bump)) break;
                    float alpha = 1.f;
                    if (bump) {
                        alpha = (m_used == -INFINITY) ? 0.f : fast_exp2(m_used - mx);
                        m_used = mx;
                        l_run *= alpha;
                    }
                    if (j > 0) {
                        // PV of the previous tile has completed (its commit precedes s_full), so O is stable
                        float o[32];
#pragma unroll 1
                        for (int c = 0; c < HD / 32; ++c) {
                            tmem_ld32(t_o + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= alpha;
                            tmem_st32(t_o + c * 32, o);
                        }
                    }
                }
                l_run += psum;
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(&sh.p_full[t]);
            }

            // ---- epilogue: O / l -> bf16 -> global ---------------------------------------------------
            ph += n_tiles;
            if constexpr (kStreaming) mbar_wait(&sh.o_full[t], n_done & 1, &sh, p.status);
            else mbar_wait(&sh.o_full[0], k & 1, &sh, p.status);
            ++n_done;
            tc_fence_after();
            const float inv = 1.f / l_run;
            // The warp stages 16 of its 32 rows at a time in its 4 KB of shared memory (16-byte pieces
            // XOR-swizzled by row) and writes them out with every 256-byte row covered by 16
            // consecutive lanes, instead of one lane per row.  (The Q buffers are not used for this:
            // the producer may already be loading the next item's Q.)
            // (at head_dim 64 a row is 128 bytes: 8 pieces, 8 lanes per row)
            constexpr int kPieces = HD / 8;                    // 16-byte pieces of an output row
            constexpr int kRowB = HD * 2;
            const uint32_t stage = sm_epi + (uint32_t)(warp * 4096);
            const int piece_r = lane % kPieces, half_r = lane / kPieces;
            const long long row0 = (long long)p.tok_off[b] + r0 + quarter * 32;
            __nv_bfloat16* obase = p.out + (long long)(p.q_head0 + hg * p.G + g0 + t) * HD + piece_r * 8;
            if constexpr (kStreaming) {
              // the thread's whole row leaves tensor memory once, scaled and rounded into kPieces 16-byte pieces
              uint32_t w[HD / 2];
              {
                  float o[HD];
                  if constexpr (HD == 128) {
                      tmem_ld128(t_o, o);
                  } else {
#pragma unroll
                      for (int c = 0; c < HD / 32; ++c) tmem_ld32(t_o + c * 32, o + c * 32);
                  }
                  tmem_wait_ld();
#pragma unroll
                  for (int i = 0; i < HD / 2; ++i) w[i] = pack_bf16(o[2 * i] * inv, o[2 * i + 1] * inv);
              }
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                  if ((lane >> 4) == h) {
#pragma unroll
                      for (int piece = 0; piece < kPieces; ++piece)
                          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                       ::"r"(stage + (lane & 15) * kRowB + ((piece ^ (lane & (kPieces - 1))) << 4)),
                                         "r"(w[4 * piece]), "r"(w[4 * piece + 1]), "r"(w[4 * piece + 2]), "r"(w[4 * piece + 3])
                                       : "memory");
                  }
                  __syncwarp();
#pragma unroll 4
                  for (int i = 0; i < kPieces / 2; ++i) {
                      const int sr = (32 / kPieces) * i + half_r;            // row inside the staged 16
                      const int lr = 16 * h + sr;                            // row inside the warp's 32
                      uint32_t w0, w1, w2, w3;
                      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                                   : "r"(stage + sr * kRowB + ((piece_r ^ (sr & (kPieces - 1))) << 4)) : "memory");
                      if (r0 + quarter * 32 + lr < C)
                          *reinterpret_cast<uint4*>(obase + (row0 + lr) * p.tok_stride) = make_uint4(w0, w1, w2, w3);
                  }
                  __syncwarp();
              }
            } else {
#pragma unroll 1
              for (int h = 0; h < 2; ++h) {
#pragma unroll 1
                  for (int c = 0; c < HD / 32; ++c) {
                      float o[32];
                      tmem_ld32(t_o + c * 32, o);
                      tmem_wait_ld();
                      if ((lane >> 4) == h) {
#pragma unroll
                          for (int i = 0; i < 4; ++i) {
                              const uint32_t w0 = pack_bf16(o[8 * i + 0] * inv, o[8 * i + 1] * inv);
                              const uint32_t w1 = pack_bf16(o[8 * i + 2] * inv, o[8 * i + 3] * inv);
                              const uint32_t w2 = pack_bf16(o[8 * i + 4] * inv, o[8 * i + 5] * inv);
                              const uint32_t w3 = pack_bf16(o[8 * i + 6] * inv, o[8 * i + 7] * inv);
                              const uint32_t piece = (uint32_t)(c * 4 + i);
                              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                           ::"r"(stage + (lane & 15) * kRowB + ((piece ^ (lane & (kPieces - 1))) << 4)),
                                             "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
                          }
                      }
                  }
                  __syncwarp();
#pragma unroll 4
                  for (int i = 0; i < kPieces / 2; ++i) {
                      const int sr = (32 / kPieces) * i + half_r;            // row inside the staged 16
                      const int lr = 16 * h + sr;                            // row inside the warp's 32
                      uint32_t w0, w1, w2, w3;
                      asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(w0), "=r"(w1), "=r"(w2), "=r"(w3)
                                   : "r"(stage + sr * kRowB + ((piece_r ^ (sr & (kPieces - 1))) << 4)) : "memory");
                      if (r0 + quarter * 32 + lr < C)
                          *reinterpret_cast<uint4*>(obase + (row0 + lr) * p.tok_stride) = make_uint4(w0, w1, w2, w3);
                  }
                  __syncwarp();
              }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kWarpTma) {
        // every TMA load this CTA issued has been consumed (the MMA warp waited on each full
        // barrier), and every MMA has completed (o_full); tensor memory can go back
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

// Exercises the bounded wait on its failure path without any copy or MMA in flight: one warp waits
// on a barrier of its own that nothing ever completes, the wait runs out after `polls` probes,
// records ZZ_ERR_TIMEOUT in the status word and the kernel returns normally.
__global__ void wait_probe_kernel(int* status, uint32_t polls, int* gave_up) {
    __shared__ Shared sh;
    if (threadIdx.x == 0) {
        mbar_init(&sh.q_full, 1);
        sh.poll_limit = polls;
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool ok = mbar_wait(&sh.q_full, 0, &sh, status);
        *gave_up = ok ? 0 : 1;
    }
}

}  // namespace

cudaError_t launch_wait_probe(int* status, unsigned int polls, int* gave_up, cudaStream_t s) {
    wait_probe_kernel<<<1, 32, 0, s>>>(status, polls, gave_up);
    count_launch();
    return cudaGetLastError();
}

static int g_num_sms = 0;

template <bool kPersistent, int HD>
static cudaError_t set_smem() {
    cudaError_t e = cudaFuncSetAttribute(prefill_kernel<kPersistent, HD, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(prefill_kernel<kPersistent, HD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    return e;
}

cudaError_t prefill_setup() {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = set_smem<true, 128>();
    if (e == cudaSuccess) e = set_smem<false, 128>();
    if (e == cudaSuccess) e = set_smem<true, 64>();
    if (e == cudaSuccess) e = set_smem<false, 64>();
    return e;
}

template <bool kPersistent, int HD>
static void launch_one(int grid, const PrefillParams& pp, const void* tq, const void* tk, const void* tv, const void* ta,
                       cudaStream_t s) {
    const CUtensorMap &mq = *static_cast<const CUtensorMap*>(tq), &mk = *static_cast<const CUtensorMap*>(tk),
                      &mv = *static_cast<const CUtensorMap*>(tv), &ma = *static_cast<const CUtensorMap*>(ta);
    if (pp.kind == ZZ_KIND_STREAMING) prefill_kernel<kPersistent, HD, true><<<grid, kThreads, kSmemBytes, s>>>(pp, mq, mk, mv, ma);
    else prefill_kernel<kPersistent, HD, false><<<grid, kThreads, kSmemBytes, s>>>(pp, mq, mk, mv, ma);
}

cudaError_t launch_prefill(const PrefillParams& p, const void* tq, const void* tk, const void* tv,
                           const void* ta, int n_items, cudaStream_t s) {
    PrefillParams pp = p;
    pp.n_items = n_items;
    if (p.D != 128 && p.D != 64) return cudaErrorInvalidValue;
    // persistent CTAs, one per SM (tensor memory and shared memory allow no more), when there are more items than SMs
    const bool persistent = g_num_sms > 0 && n_items > g_num_sms;
    if (p.D == 128) {
        if (persistent) launch_one<true, 128>(g_num_sms, pp, tq, tk, tv, ta, s);
        else launch_one<false, 128>(n_items, pp, tq, tk, tv, ta, s);
    } else {
        if (persistent) launch_one<true, 64>(g_num_sms, pp, tq, tk, tv, ta, s);
        else launch_one<false, 64>(n_items, pp, tq, tk, tv, ta, s);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace zz
