// KV append with sink + recent eviction, cache reset, and the head regrouping copies of the
// mixed-head layer.  All three are pure data movement: 16-byte vector loads and stores.
#include <cstring>

#include "zz_common.cuh"

namespace zz {

// One thread moves one 16-byte piece of a K row and the matching piece of the V row (a row has
// head_dim / 8 pieces).
// grid = (blocks over the work of the longest sequence, batch).
//
// Retrieval group: every new token i goes to slot len + i.
// Streaming group: token t = len + i goes to slot(t) = t (t < S) or S + ((t - S) mod W).
//   Of a chunk of C tokens only the sinks it contains and its last W tokens survive, so only
//   those are written (each surviving token owns its slot: no write races, and the result is
//   what appending the chunk token by token leaves behind).
// The length is bumped by the last block to finish, after every block has read the old one.
__global__ void __launch_bounds__(256) append_kernel(const AppendParams p) {
    const int b = blockIdx.y;
    const int C = p.n_new[b];
    const int P = p.len[b];
    const SeqDesc sd = p.desc[b];
    const int nS = p.Hkv - p.nR;
    const int n_sink = max(0, min(p.S - P, C));          // chunk tokens that are sinks
    const int tail0 = max(n_sink, C - p.W);              // first surviving non-sink chunk token
    const int n_cand = n_sink + (C - tail0);
    const int ppr = p.D >> 3;                            // 16-byte pieces per row
    const long long workR = p.skip_retrieval ? 0ll : (long long)C * p.nR * ppr;
    const long long workS = (long long)n_cand * nS * ppr;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < workR + workS) {
        int i, hi, piece, kind;
        long long slot;
        if (idx < workR) {
            kind = ZZ_KIND_RETRIEVAL;
            piece = (int)(idx % ppr);
            const long long r = idx / ppr;
            hi = (int)(r % p.nR);
            i = (int)(r / p.nR);
            slot = (long long)P + i;
        } else {
            kind = ZZ_KIND_STREAMING;
            const long long j = idx - workR;
            piece = (int)(j % ppr);
            const long long r = j / ppr;
            hi = (int)(r % nS);
            const int c = (int)(r / nS);
            i = (c < n_sink) ? c : tail0 + (c - n_sink);
            const int t = P + i;
            slot = (t < p.S) ? t : p.S + ((t - p.S) % p.W);
            if (hi == 0 && piece == 0) p.pos[(long long)b * p.ring + slot] = t;
        }
        const int src_head = p.head_list[(kind == ZZ_KIND_RETRIEVAL) ? hi : p.nR + hi];
        const long long slots_per_head = (kind == ZZ_KIND_RETRIEVAL) ? sd.cap : p.ring;
        const long long src = ((long long)(p.tok_off[b] + i) * p.Hkv + src_head) * p.D + piece * 8;
        long long dst = ((long long)hi * slots_per_head + slot) * p.D + piece * 8;
        if (kind == ZZ_KIND_RETRIEVAL && p.page_table) {
            // paged store: the slot's page comes from the table (K rows, then V rows, per page)
            const int page = p.page_table[sd.tbl + (int)(slot >> 7) * p.nR + hi];
            dst = (long long)page * kPageElems + (slot & (kPageTokens - 1)) * kD + piece * 8;
        }
        const uint4 kk = *reinterpret_cast<const uint4*>(p.k_new + src);
        const uint4 vv = *reinterpret_cast<const uint4*>(p.v_new + src);
        *reinterpret_cast<uint4*>(p.arena + sd.k_off[kind] + dst) = kk;
        *reinterpret_cast<uint4*>(p.arena + sd.v_off[kind] + dst) = vv;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int total = gridDim.x * gridDim.y;
        const unsigned int prev = atomicAdd(p.counter, 1u);
        if (prev == total - 1) {
            for (int s = 0; s < p.B; ++s) p.len[s] += p.n_new[s];
            *p.counter = 0u;
            __threadfence();
        }
    }
}

cudaError_t launch_append(const AppendParams& p, int grid_x, cudaStream_t s) {
    dim3 grid(grid_x > 0 ? grid_x : 1, p.B);
    append_kernel<<<grid, 256, 0, s>>>(p);
    count_launch();
    return cudaGetLastError();
}

// len[l][seq] = 0 and pos[l][seq][*] = -1 for one sequence (seq >= 0) or all of them.
__global__ void reset_kernel(int* len, int* pos, int L, int B, int ring, int seq) {
    const long long n_seq = (seq < 0) ? B : 1;
    const long long total = (long long)L * n_seq * (ring + 1);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int e = (int)(i % (ring + 1));
        const long long r = i / (ring + 1);
        const int b = (seq < 0) ? (int)(r % B) : seq;
        const int l = (int)(r / n_seq);
        if (e == ring) len[(long long)l * B + b] = 0;
        else pos[((long long)l * B + b) * ring + e] = -1;
    }
}

cudaError_t launch_reset(int* len, int* pos, int L, int B, int ring, int seq, cudaStream_t s) {
    reset_kernel<<<64, 256, 0, s>>>(len, pos, L, B, ring, seq);
    count_launch();
    return cudaGetLastError();
}

// Mixed-head layer: move whole query/output head rows between the model's head order
// [token][Hkv*G][128] and the compact group order (retrieval heads first, then streaming),
// 16 bytes per thread.
__global__ void __launch_bounds__(256) regroup_kernel(const GatherParams p) {
    // launched with programmatic stream serialization: the launch itself overlaps the previous
    // kernel's tail, the data dependence is kept by waiting here before anything is read
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int ppr = p.D >> 3;
    const long long total = p.tokens * p.Hkv * p.G * ppr;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int piece = (int)(i % ppr);
        long long r = i / ppr;
        const int g = (int)(r % p.G);
        r /= p.G;
        const int c = (int)(r % p.Hkv);   // compact KV-head index
        long long tok = r / p.Hkv;
        const int* hl = p.head_list;
        if (p.layer_ids) {
            const int layer = p.layer_ids[tok / p.toks_per_layer];
            tok = (long long)layer * p.toks_per_layer + tok % p.toks_per_layer;
            hl += (long long)layer * p.Hkv;
        }
        const int h = hl[c];              // model KV-head index
        const long long compact = ((tok * p.Hkv + c) * p.G + g) * p.D + piece * 8;
        const long long model = ((tok * p.Hkv + h) * p.G + g) * p.D + piece * 8;
        if (p.to_compact)
            *reinterpret_cast<uint4*>(p.dst + compact) = *reinterpret_cast<const uint4*>(p.src + model);
        else
            *reinterpret_cast<uint4*>(p.dst + model) = *reinterpret_cast<const uint4*>(p.src + compact);
    }
}

// Page-table entries of newly allocated pages (at most 480 per launch, passed by value).
__global__ void __launch_bounds__(512) table_update_kernel(int* table, const TableUpdate u) {
    const int i = threadIdx.x;
    if (i < u.n) table[u.idx[i]] = u.val[i];
}

cudaError_t launch_table_update(int* table, const TableUpdate& u, cudaStream_t s) {
    table_update_kernel<<<1, 512, 0, s>>>(table, u);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_regroup(const GatherParams& p, cudaStream_t s, int programmatic) {
    const long long total = p.tokens * p.Hkv * p.G * (p.D >> 3);
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, regroup_kernel, p);
    count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace zz
