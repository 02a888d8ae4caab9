// gsd_unmerge_tree: the token graph reverted to a tree for verification (Sec. 5.4, Fig. 4: the
// successors of every redundant node are replicated from the node it was merged into, and the
// tree is verified as in tree-structured decoding).  On the verification DAG (parent lists in
// CSR form) this is the unfolding from the root: one tree node per root path, numbered level by
// level, inside a level by (tree index of the parent, id of the copied node).
//
// One CTA per sequence.  The child lists of the DAG are built in shared memory (degree count,
// scan, fill, a short insertion sort per list for the ascending order); then the tree grows one
// level per round: the nodes of the last level look up the degree of the node they copy, a
// block-wide exclusive scan over the level gives every node the slot of its first child, and
// the children are written behind the level.  Growth stops at the depth limit, when a level
// comes out empty, or when the capacity is reached (the prefix of the level order is kept).
#include "gsd_internal.cuh"

namespace gsd {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxEdges = GSD_UNMERGE_MAX_EDGES;

__device__ __forceinline__ int block_exclusive_scan(int x, int* s_warp, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();                      // s_warp may still be read from the previous call
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    int base = 0, sum = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
        if (w < warp) base += s_warp[w];
        sum += s_warp[w];
    }
    total = sum;
    return base + inc - x;
}

__global__ void __launch_bounds__(kThreads)
unmerge_kernel(const int32_t* tok_all, const int32_t* pptr_all, const int32_t* pidx_all, int32_t* tt_all,
               int32_t* tp_all, int32_t* ts_all, int32_t* count_all, int N, int Ecap, int Ucap, int max_depth,
               int32_t* status) {
    __shared__ int s_ptr[GSD_MAX_NODES + 1];     // sanitised parent row pointers
    __shared__ int s_deg[GSD_MAX_NODES];         // children per node
    __shared__ int s_cptr[GSD_MAX_NODES + 1];
    __shared__ int s_fill[GSD_MAX_NODES];
    __shared__ short s_child[kMaxEdges];
    __shared__ int s_tok[GSD_MAX_NODES];
    __shared__ int s_warp[kThreads / 32];
    const int b = blockIdx.x, tid = threadIdx.x;
    const int32_t* tok = tok_all + (size_t)b * N;
    const int32_t* pptr = pptr_all + (size_t)b * (N + 1);
    const int32_t* pidx = pidx_all + (size_t)b * Ecap;
    int32_t* tt = tt_all + (size_t)b * Ucap;
    int32_t* tp = tp_all + (size_t)b * Ucap;
    int32_t* ts = ts_all + (size_t)b * Ucap;
    unsigned flags = 0;
    const int ecap = min(Ecap, kMaxEdges);

    for (int v = tid; v <= N; v += kThreads) {
        int e = pptr[v];
        if (e < 0 || e > ecap) {
            flags |= GSD_DEV_BAD_CSR;
            e = e < 0 ? 0 : ecap;
        }
        s_ptr[v] = e;
    }
    for (int v = tid; v < N; v += kThreads) {
        s_deg[v] = 0;
        s_fill[v] = 0;
        s_tok[v] = tok[v];
    }
    __syncthreads();
    {
        // row pointers that do not start at zero or go backwards: running maximum, as in gsd_accept
        int bad = 0;
        for (int v = tid; v < N; v += kThreads) bad |= (s_ptr[v] > s_ptr[v + 1]);
        if (tid == 0 && s_ptr[0] != 0) bad = 1;
        if (__syncthreads_or(bad)) {
            flags |= GSD_DEV_BAD_CSR;
            if (tid == 0) {
                int run = 0;
                s_ptr[0] = 0;
                for (int v = 1; v <= N; ++v) {
                    run = max(run, s_ptr[v]);
                    s_ptr[v] = run;
                }
            }
            __syncthreads();
        }
    }
    // an edge counts once: a parent index outside [0, v) or listed again in the same row is skipped
    auto edge_ok = [&](int v, int e, int p) -> bool {
        if (p < 0 || p >= v) return false;
        for (int f = s_ptr[v]; f < e; ++f)
            if (pidx[f] == p) return false;
        return true;
    };
    for (int v = tid; v < N; v += kThreads)
        for (int e = s_ptr[v]; e < s_ptr[v + 1]; ++e) {
            const int p = pidx[e];
            if (edge_ok(v, e, p)) atomicAdd(&s_deg[p], 1);
            else if (p < 0 || p >= v) flags |= GSD_DEV_BAD_CSR;
        }
    __syncthreads();
    {
        // exclusive scan of the degrees (N <= 512: two entries per thread)
        const int v0 = 2 * tid, v1 = 2 * tid + 1;
        const int d0 = v0 < N ? s_deg[v0] : 0, d1 = v1 < N ? s_deg[v1] : 0;
        int total;
        const int off = block_exclusive_scan(d0 + d1, s_warp, total);
        if (v0 < N) s_cptr[v0] = off;
        if (v1 < N) s_cptr[v1] = off + d0;
        if (tid == 0) s_cptr[N] = total;
    }
    __syncthreads();
    for (int v = tid; v < N; v += kThreads)
        for (int e = s_ptr[v]; e < s_ptr[v + 1]; ++e) {
            const int p = pidx[e];
            if (edge_ok(v, e, p)) s_child[s_cptr[p] + atomicAdd(&s_fill[p], 1)] = (short)v;
        }
    __syncthreads();
    for (int p = tid; p < N; p += kThreads) {       // children in ascending order
        const int lo = s_cptr[p], hi = s_cptr[p + 1];
        for (int i = lo + 1; i < hi; ++i) {
            const short x = s_child[i];
            int j = i - 1;
            while (j >= lo && s_child[j] > x) {
                s_child[j + 1] = s_child[j];
                --j;
            }
            s_child[j + 1] = x;
        }
    }
    if (tid == 0) {
        tt[0] = s_tok[0];
        tp[0] = -1;
        ts[0] = 0;
    }
    __syncthreads();

    int lvl_begin = 0, lvl_end = 1;
    bool overflow = false;
    for (int depth = 0; depth < max_depth && lvl_end > lvl_begin && !overflow; ++depth) {
        int base = 0;                                // children of this level created so far
        for (int c = lvl_begin; c < lvl_end; c += kThreads) {
            const int u = c + tid;
            const int src = u < lvl_end ? ts[u] : -1;
            const int deg = src >= 0 ? s_deg[src] : 0;
            int total;
            const int off = block_exclusive_scan(deg, s_warp, total);
            const int first = lvl_end + base + off;
            for (int j = 0; j < deg; ++j) {
                const int idx = first + j;
                if (idx >= Ucap) break;
                const int child = s_child[s_cptr[src] + j];
                if (!GSD_IN_BOUNDS(child > src && child < N && s_cptr[src] + j < kMaxEdges, status)) continue;
                tt[idx] = s_tok[child];
                tp[idx] = u;
                ts[idx] = child;
            }
            base += total;
        }
        overflow = lvl_end + base > Ucap;            // (a level that fills the capacity exactly goes on:
        if (overflow) flags |= GSD_DEV_TREE_FULL;    //  its own children, if any, raise the flag next round)
        lvl_begin = lvl_end;
        lvl_end = min(lvl_end + base, Ucap);
        __syncthreads();                             // the new level's entries are read next round
    }
    // the depth limit or the capacity may have cut the tree: say so only for the capacity
    for (int i = lvl_end + tid; i < Ucap; i += kThreads) tt[i] = tp[i] = ts[i] = -1;
    if (tid == 0) count_all[b] = lvl_end;
    if (flags && status) atomicOr((unsigned*)status, flags);
}

}  // namespace
}  // namespace gsd

extern "C" int gsd_unmerge_tree(const int32_t* draft_tokens, const int32_t* parent_ptr, const int32_t* parent_idx,
                                int32_t* tree_tokens, int32_t* tree_parent, int32_t* tree_source,
                                int32_t* tree_count, int32_t B, int32_t N, int32_t Ecap, int32_t Ucap,
                                int32_t max_depth, int32_t* status, void* stream) {
    using namespace gsd;
    if (!draft_tokens || !parent_ptr || !parent_idx || !tree_tokens || !tree_parent || !tree_source || !tree_count)
        return GSD_ERR_NULL_POINTER;
    if (B < 1 || B > 65535 * 32 || N < 1 || N > GSD_MAX_NODES || Ecap < 1 || Ucap < 1 || max_depth < 0)
        return GSD_ERR_BAD_SHAPE;
    unmerge_kernel<<<B, kThreads, 0, (cudaStream_t)stream>>>(draft_tokens, parent_ptr, parent_idx, tree_tokens,
                                                             tree_parent, tree_source, tree_count, N, Ecap, Ucap,
                                                             max_depth, status);
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}
