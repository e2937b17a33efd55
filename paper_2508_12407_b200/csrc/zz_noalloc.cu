// Decode attention for callers that must not allocate device memory.
//
// Some callers of this library run where cudaMalloc is off limits: inside a serving loop that
// has handed every byte of the device to its own pool, or in a plug-in whose host forbids driver
// allocations after start-up.  The regular
// path asks such a caller for a workspace (zz_cache_query / zz_cache_create); this entry point
// asks for nothing but the inputs and the output.  The split-sequence decode kernel still needs
// scratch memory (per-split partial outputs, their softmax statistics, the arrival counters and
// the device copy of the lengths), so that scratch lives in a fixed array in the library's own
// device image.  Every GPU that loads the library carries the array until the process exits.
#include <cstring>

#include "zz_common.cuh"

namespace {

constexpr int kStaticMaxRows = 64;       // batch * n_q_heads
constexpr int kStaticMaxSplits = 64;
constexpr int kStaticMaxBatch = 16;
// layout of the scratch, in bytes
constexpr size_t kOffCounters = 0;                                    // (pairs + batch) uint32, zeroed per call
constexpr size_t kCountersBytes = 1024;
constexpr size_t kOffLen = kOffCounters + kCountersBytes;             // batch int32
constexpr size_t kOffStatus = kOffLen + 256;                          // status word
constexpr size_t kOffPartMl = kOffStatus + 256;                       // rows * splits * 2 float
constexpr size_t kPartMlBytes = (size_t)kStaticMaxRows * kStaticMaxSplits * 2 * sizeof(float);
constexpr size_t kOffPartO = kOffPartMl + kPartMlBytes;               // rows * splits * 128 float
constexpr size_t kPartOBytes = (size_t)kStaticMaxRows * kStaticMaxSplits * zz::kD * sizeof(float);
constexpr size_t kScratchBytes = kOffPartO + kPartOBytes;             // about 2.1 MB

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// calls, never an address a kernel could use.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch on the current device, looked up once per device.
int scratch_for_current_device(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ZZ_ERR_CUDA;
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return ZZ_ERR_CUDA;
        if (zz::decode_setup() != cudaSuccess) return ZZ_ERR_CUDA;
        g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_ptr[dev];
    return ZZ_OK;
}

}  // namespace

extern "C" int zz_decode_attn_static(const void* d_q, const void* d_k, const void* d_v, void* d_out,
                                     const int32_t* h_len, int32_t batch, int32_t n_q_heads,
                                     int32_t n_kv_heads, int32_t capacity, float softmax_scale, void* stream) {
    if (!d_q || !d_k || !d_v || !d_out || !h_len) return ZZ_ERR_INVALID_ARG;
    if (((uintptr_t)d_q | (uintptr_t)d_k | (uintptr_t)d_v | (uintptr_t)d_out) & 15) return ZZ_ERR_INVALID_ARG;
    if (batch < 1 || n_q_heads < 1 || n_kv_heads < 1 || capacity < 1 || !(softmax_scale > 0.f))
        return ZZ_ERR_INVALID_ARG;
    if (n_q_heads % n_kv_heads != 0 || n_q_heads / n_kv_heads > 16) return ZZ_ERR_UNSUPPORTED;
    // the fixed scratch bounds the problem: say so instead of overrunning it
    if (batch > kStaticMaxBatch || (long long)batch * n_q_heads > kStaticMaxRows) return ZZ_ERR_WORKSPACE;
    for (int b = 0; b < batch; ++b)
        if (h_len[b] < 1 || h_len[b] > capacity) return ZZ_ERR_INVALID_ARG;

    unsigned char* scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != ZZ_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const int G = n_q_heads / n_kv_heads;
    zz::DecodeParams p;
    memset(&p, 0, sizeof p);
    // the stores are the caller's tensors: K and V as [batch][n_kv_heads][capacity][128]
    __nv_bfloat16* kbase = static_cast<__nv_bfloat16*>(const_cast<void*>(d_k));
    // V is addressed relative to K's base (both are 16-byte aligned, so the distance is a whole
    // number of elements)
    const long long v_minus_k = ((long long)(intptr_t)d_v - (long long)(intptr_t)d_k) / 2;
    p.arena = kbase;
    for (int b = 0; b < batch; ++b) {
        const long long off = (long long)b * n_kv_heads * capacity * zz::kD;
        p.sd[b].k_off[ZZ_KIND_RETRIEVAL] = off;
        p.sd[b].v_off[ZZ_KIND_RETRIEVAL] = v_minus_k + off;
        p.sd[b].cap = capacity;
    }
    p.len = reinterpret_cast<int*>(scratch + kOffLen);
    p.q = static_cast<const __nv_bfloat16*>(d_q);
    p.out = static_cast<__nv_bfloat16*>(d_out);
    p.q_tok_stride = (long long)n_q_heads * zz::kD;
    p.q_head0 = 0;
    p.part_o = reinterpret_cast<float*>(scratch + kOffPartO);
    p.part_ml = reinterpret_cast<float*>(scratch + kOffPartMl);
    p.counters = reinterpret_cast<unsigned int*>(scratch + kOffCounters);
    p.seq_counters = p.counters + (size_t)batch * n_kv_heads;
    p.status = reinterpret_cast<int*>(scratch + kOffStatus);
    p.kind = ZZ_KIND_RETRIEVAL;
    p.D = zz::kD;
    p.ring = 1;
    p.Hg = n_kv_heads;
    p.G = G;
    p.B = batch;
    p.max_splits = kStaticMaxSplits;
    p.scale_log2 = softmax_scale * 1.4426950408889634f;
    p.n_kv_total = n_kv_heads;

    // split plan: 4-warp CTAs, about two per SM, never more than the scratch has room for
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return ZZ_ERR_CUDA;
    }
    long long total = 0;
    for (int b = 0; b < batch; ++b) total += h_len[b];
    const int slots = 2 * sms;
    long long per = (total * n_kv_heads + slots - 1) / slots;
    if (per < 256) per = 256;
    for (;;) {
        long long items = 0;
        int worst = 0;
        for (int b = 0; b < batch; ++b) {
            const int s = (int)((h_len[b] + per - 1) / per);
            items += (long long)s * n_kv_heads;
            if (s > worst) worst = s;
        }
        if ((items <= slots || per >= total) && worst <= kStaticMaxSplits) break;
        per += 16;
    }
    p.split_start[0] = 0;
    for (int b = 0; b < batch; ++b) {
        const int s = (int)((h_len[b] + per - 1) / per);
        p.chunk[b] = (h_len[b] + s - 1) / s;
        p.split_start[b + 1] = p.split_start[b] + s;
    }
    const int items = p.split_start[batch] * n_kv_heads;

    // the array keeps whatever the previous call left: counters must start at zero
    if (cudaMemsetAsync(scratch + kOffCounters, 0, kCountersBytes, st) != cudaSuccess) return ZZ_ERR_CUDA;
    if (cudaMemcpyAsync(scratch + kOffLen, h_len, (size_t)batch * sizeof(int32_t), cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
        return ZZ_ERR_CUDA;
    return zz::launch_decode(p, items, 4, st) == cudaSuccess ? ZZ_OK : ZZ_ERR_CUDA;
}

extern "C" int zz_decode_attn_static_limits(int32_t* max_batch, int32_t* max_batch_times_q_heads,
                                            size_t* scratch_bytes) {
    if (!max_batch || !max_batch_times_q_heads || !scratch_bytes) return ZZ_ERR_INVALID_ARG;
    *max_batch = kStaticMaxBatch;
    *max_batch_times_q_heads = kStaticMaxRows;
    *scratch_bytes = kScratchBytes;
    return ZZ_OK;
}
