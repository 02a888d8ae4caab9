// gsd_commit_kv: append the draft K/V rows of the accepted path to the KV cache and advance
// the sequence lengths (the cache update after verification: "Others" in the paper's time
// breakdown, Sec. 7.1 / Table 3; KV caching, Sec. 4.2).
//
// One CTA per sequence: it reads the old length once, copies up to accepted_len[b] rows of
// Hkv*D bf16 for K and for V with 16-byte loads/stores, and only then writes the new length,
// so the update is safe in place.  The data is a few KB per sequence: the call is bound by
// launch and memory latency, not by bandwidth.
#include "gsd_internal.cuh"

namespace gsd {
namespace {

constexpr int kThreads = 256;

struct CommitArgs {
    uint4* k_cache;
    uint4* v_cache;
    const uint4* draft_k;
    const uint4* draft_v;
    const int32_t* nodes;
    const int32_t* len;
    int32_t* seq_lens;
    int32_t* status;
    int N, Lmax, Tcap;
    int row16;   // 16-byte chunks per (position, all kv heads) row = Hkv * D * 2 / 16
};

__global__ void __launch_bounds__(kThreads) commit_kernel(CommitArgs a) {
    const int b = blockIdx.x;
    __shared__ int s_src[GSD_MAX_NODES];   // source node of each destination position
    __shared__ int s_count;
    int L = a.seq_lens[b];
    unsigned flags = 0;
    if (L < 0 || L > a.Lmax) {
        flags |= GSD_DEV_BAD_SEQ_LEN;
        L = L < 0 ? 0 : a.Lmax;
    }
    {
        // compact the valid node ids in path order: every thread reads one entry, the positions
        // come from warp ballots and a scan over the warp totals
        __shared__ int s_warp_tot[kThreads / 32];
        int len = a.len[b];
        if (len > a.Tcap) len = a.Tcap;
        if (len > GSD_MAX_NODES) len = GSD_MAX_NODES;
        if (threadIdx.x == 0) s_count = 0;
        int base = 0;
        for (int i0 = 0; i0 < len; i0 += kThreads) {      // one pass unless Tcap > 256
            const int i = i0 + threadIdx.x;
            int node = -1;
            bool valid = false;
            if (i < len) {
                node = a.nodes[(size_t)b * a.Tcap + i];
                valid = node >= 0 && node < a.N;
                if (!valid) flags |= GSD_DEV_BAD_CSR;
            }
            const unsigned vote = __ballot_sync(0xFFFFFFFFu, valid);
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            if (lane == 0) s_warp_tot[warp] = __popc(vote);
            __syncthreads();
            int before = base;
            for (int w = 0; w < warp; ++w) before += s_warp_tot[w];
            const int pos = before + __popc(vote & ((1u << lane) - 1u));
            if (valid) {
                if (L + pos < a.Lmax) s_src[pos] = node;
                else flags |= GSD_DEV_CACHE_FULL;
            }
            int total = 0;
            for (int w = 0; w < kThreads / 32; ++w) total += s_warp_tot[w];
            base += total;
            __syncthreads();
        }
        if (threadIdx.x == 0) s_count = min(base, a.Lmax - L);
        if (flags && a.status) atomicOr((unsigned*)a.status, flags);
    }
    __syncthreads();
    const int n = s_count;
    const long total = (long)n * a.row16;
    for (long t = threadIdx.x; t < total; t += kThreads) {
        const int i = (int)(t / a.row16), ch = (int)(t % a.row16);
        if (!GSD_IN_BOUNDS(s_src[i] >= 0 && s_src[i] < a.N && L + i < a.Lmax, a.status)) continue;
        const size_t src = ((size_t)b * a.N + s_src[i]) * a.row16 + ch;
        const size_t dst = ((size_t)b * a.Lmax + L + i) * a.row16 + ch;
        a.k_cache[dst] = a.draft_k[src];
        a.v_cache[dst] = a.draft_v[src];
    }
    __syncthreads();
    if (threadIdx.x == 0) a.seq_lens[b] = L + n;
}

}  // namespace
}  // namespace gsd

extern "C" int gsd_commit_kv(void* k_cache, void* v_cache, const void* draft_k, const void* draft_v,
                             const int32_t* accepted_nodes, const int32_t* accepted_len,
                             int32_t* seq_lens, const gsd_commit_params* p, int32_t* status,
                             void* stream) {
    using namespace gsd;
    if (!p || !k_cache || !v_cache || !draft_k || !draft_v || !accepted_nodes || !accepted_len || !seq_lens)
        return GSD_ERR_NULL_POINTER;
    if (p->B < 1 || p->N < 1 || p->N > GSD_MAX_NODES || p->Hkv < 1 || p->D < 8 || p->D % 8 != 0 ||
        p->Lmax < 1 || p->Tcap < 1 || p->B > 65535 * 32)
        return GSD_ERR_BAD_SHAPE;
    const void* ptrs[] = {k_cache, v_cache, draft_k, draft_v};
    for (const void* ptr : ptrs)
        if (((uintptr_t)ptr & 15u) != 0) return GSD_ERR_MISALIGNED;
    CommitArgs a;
    a.k_cache = (uint4*)k_cache; a.v_cache = (uint4*)v_cache;
    a.draft_k = (const uint4*)draft_k; a.draft_v = (const uint4*)draft_v;
    a.nodes = accepted_nodes; a.len = accepted_len; a.seq_lens = seq_lens; a.status = status;
    a.N = p->N; a.Lmax = p->Lmax; a.Tcap = p->Tcap;
    a.row16 = p->Hkv * p->D * 2 / 16;
    commit_kernel<<<p->B, kThreads, 0, (cudaStream_t)stream>>>(a);
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}
