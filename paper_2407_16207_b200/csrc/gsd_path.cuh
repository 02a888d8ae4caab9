// Longest accepted root path through the draft DAG (Sec. 4.1 longest-path selection; Sec. 3
// rejection cascade), shared by the deterministic and the non-deterministic verification.
// One CTA of kPathThreads threads per sequence.  The caller supplies the test of one step
// parent -> v; this file does the rest: parent lists on chip, level-synchronous relaxation of
// best[v] = 1 + max over accepted steps into v, choice of the end node (longest, then lowest
// index), walk back (lowest predecessor that carries length - 1), emission of the path's node
// ids and drafted tokens.  The token the target model contributes at the end is the caller's.
//
// The pass runs on one SM while the rest of the device may already be idle, so it is laid out
// for few dependent trips to memory: tokens, row pointers and the parent indices are fetched in
// one go; the relaxation costs one barrier per round (two copies of best[]); every node picks
// its predecessor in parallel, after which the walk back is a pointer chase in shared memory
// and the outputs are written by the whole block.
#pragma once
#include "gsd_internal.cuh"

namespace gsd {

constexpr int kPathThreads = 256;
constexpr int kPathNone = 0x7FFFFFFF;
constexpr int kPathNodeSlots = (GSD_MAX_NODES + kPathThreads - 1) / kPathThreads;
constexpr int kPathEdgeCache = 3 * GSD_MAX_NODES;   // parent edges of one sequence kept in shared memory
static_assert(kPathEdgeCache % kPathThreads == 0, "the edge prefetch is dealt out in whole rounds");

struct PathIo {
    const int32_t* tok;     // [N] drafted tokens of the sequence
    const int32_t* pptr;    // [N+1]
    const int32_t* pidx;    // [Ecap]
    int32_t* out_tok;       // [Tcap]
    int32_t* out_nodes;     // [Tcap] or nullptr
    int32_t* out_len;       // one entry
    int32_t* status;        // device status word or nullptr
    int N, V, Ecap, Tcap;
};

struct PathResult {
    int edges;           // m: the accepted path has m + 1 nodes
    int end;             // its last node
    bool end_has_child;  // some node lists `end` as a parent (only filled in with kCacheOutcome)
};

// The test of a step p -> v comes in two halves: `edge_pre(p, v)` fetches what the test needs
// from global memory (a float), `step_ok(pre, p, v)` decides.  With kCacheOutcome both are
// called once per step when the parent lists fit the on-chip cache (one thread per step, all at
// once - for tests that touch global memory); otherwise they are called again on every use (for
// tests that cost a comparison).  Between the two halves the function calls `mid()` (all
// threads; it returns status bits) and meets at a barrier: a caller whose decision needs results
// of an earlier kernel waits for them there, AFTER the graph and the values of `edge_pre` have
// been fetched.  `flags` carries status bits the caller has already found; the function adds its
// own and publishes them.  All threads of the CTA must call it; all return the same result.
// out_tok[edges] is left for the caller, entries past it are set to -1.
template <bool kCacheOutcome, class StepOk, class EdgePre, class Mid>
__device__ PathResult longest_accepted_path_ex(const PathIo& io, unsigned flags, StepOk step_ok, EdgePre edge_pre, Mid mid) {
    __shared__ int s_best[2][GSD_MAX_NODES];      // two copies: a round reads one and writes the other
    __shared__ int s_tok[GSD_MAX_NODES];
    __shared__ int s_ptr[GSD_MAX_NODES + 1];
    __shared__ int s_edge[kPathEdgeCache];
    __shared__ unsigned char s_eok[kPathEdgeCache];
    __shared__ float s_eval[kCacheOutcome ? kPathEdgeCache : 1];   // what edge_pre fetched for each step
    __shared__ short s_enode[kPathEdgeCache];   // the node a step leads into
    __shared__ short s_path[GSD_MAX_NODES];     // the chosen path, root first
    __shared__ int s_red[kPathThreads / 32];
    __shared__ unsigned s_flags;
    __shared__ int s_m, s_end;
    const int N = io.N, tid = threadIdx.x;
    if (tid == 0) s_flags = 0;
    // tokens, row pointers and (speculatively: the row holds Ecap entries whatever the pointers
    // say) the parent indices, all in one trip to memory
    // (every load is issued before the first of them is used: the loops below have constant
    // trip counts and are unrolled, so the three arrays cost one round trip, not three)
    const int n_prefetch = min(io.Ecap, kPathEdgeCache);
    int r_tok[kPathNodeSlots], r_ptr[kPathNodeSlots + 1], r_edge[kPathEdgeCache / kPathThreads];
#pragma unroll
    for (int k = 0; k < kPathNodeSlots; ++k) r_tok[k] = tid + k * kPathThreads < N ? io.tok[tid + k * kPathThreads] : 0;
#pragma unroll
    for (int k = 0; k <= kPathNodeSlots; ++k) r_ptr[k] = tid + k * kPathThreads <= N ? io.pptr[tid + k * kPathThreads] : 0;
#pragma unroll
    for (int k = 0; k < kPathEdgeCache / kPathThreads; ++k)
        r_edge[k] = tid + k * kPathThreads < n_prefetch ? io.pidx[tid + k * kPathThreads] : 0;
#pragma unroll
    for (int k = 0; k < kPathNodeSlots; ++k) {
        const int v = tid + k * kPathThreads;
        if (v < N) {
            s_tok[v] = r_tok[k];
            if (r_tok[k] < 0 || r_tok[k] >= io.V) flags |= GSD_DEV_BAD_TOKEN;
            s_best[0][v] = v == 0 ? 0 : -1;
        }
    }
#pragma unroll
    for (int k = 0; k <= kPathNodeSlots; ++k) {
        const int v = tid + k * kPathThreads;
        if (v <= N) {
            int e = r_ptr[k];
            if (e < 0 || e > io.Ecap) {
                flags |= GSD_DEV_BAD_CSR;
                e = e < 0 ? 0 : io.Ecap;
            }
            s_ptr[v] = e;
        }
    }
#pragma unroll
    for (int k = 0; k < kPathEdgeCache / kPathThreads; ++k)
        if (tid + k * kPathThreads < n_prefetch) s_edge[tid + k * kPathThreads] = r_edge[k];
    __syncthreads();
    // Row pointers must start at zero and never decrease.  Otherwise they are replaced by their
    // running maximum (a row whose pointer goes backwards becomes empty, the rows stay disjoint
    // and every edge below the last pointer has exactly one owner) and the status bit is set.
    {
        int bad = 0;
        for (int v = tid; v < N; v += kPathThreads) bad |= (s_ptr[v] > s_ptr[v + 1]);
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
    // the relaxation rounds walk the parent lists again and again: keep them, and the outcome
    // of every step, on chip
    const int n_edges = s_ptr[N];
    const bool cached = n_edges <= kPathEdgeCache;
    if (cached && kCacheOutcome) {
        for (int v = tid; v < N; v += kPathThreads)
            for (int e = s_ptr[v]; e < s_ptr[v + 1]; ++e) s_enode[e] = (short)v;
        __syncthreads();
        for (int e = tid; e < n_edges; e += kPathThreads) {
            const int p = s_edge[e], v = s_enode[e];
            s_eval[e] = (p >= 0 && p < v && s_tok[v] >= 0 && s_tok[v] < io.V) ? edge_pre(p, v) : 0.f;
        }
    }
    flags |= mid();
    __syncthreads();
    if (cached && kCacheOutcome) {
        for (int e = tid; e < n_edges; e += kPathThreads) {
            const int p = s_edge[e], v = s_enode[e];
            s_eok[e] = (p >= 0 && p < v && s_tok[v] >= 0 && s_tok[v] < io.V) ? (unsigned char)step_ok(s_eval[e], p, v) : 0;
        }
        __syncthreads();
    }
    auto parent_at = [&](int e) -> int { return cached ? s_edge[e] : io.pidx[e]; };
    auto ok_at = [&](int e, int p, int v) -> bool {
        if (cached && kCacheOutcome) return s_eok[e] != 0;
        return s_tok[v] >= 0 && s_tok[v] < io.V && step_ok(edge_pre(p, v), p, v);
    };

    // level-synchronous relaxation: after round r every node whose longest accepted root
    // path has <= r edges is final; values only grow, so it stops when nothing changed
    int cur_buf = 0;
    for (int round = 0; round < N; ++round) {
        const int* rd = s_best[cur_buf];
        int* wr = s_best[cur_buf ^ 1];
        int changed = 0;
#pragma unroll
        for (int k = 0; k < kPathNodeSlots; ++k) {
            const int v = tid + k * kPathThreads;
            if (v < N) {
                int cur = rd[v];
                if (v > 0) {
                    for (int e = s_ptr[v]; e < s_ptr[v + 1]; ++e) {
                        const int p = parent_at(e);
                        if (p < 0 || p >= v) {
                            flags |= GSD_DEV_BAD_CSR;
                            continue;
                        }
                        const int bp = rd[p];
                        if (bp >= 0 && bp + 1 > cur && ok_at(e, p, v)) cur = bp + 1;
                    }
                }
                wr[v] = cur;
                changed |= (cur != rd[v]);
            }
        }
        cur_buf ^= 1;
        if (!__syncthreads_or(changed)) break;
    }
    const int* best = s_best[cur_buf];
    int* pred = s_best[cur_buf ^ 1];   // the other copy now takes every node's predecessor on its best path
    __syncthreads();                   // (every thread has left the last round's reads of it)

    // every node: the lowest predecessor with an accepted step that carries length - 1
    int key = -1;
    for (int v = tid; v < N; v += kPathThreads) {
        const int bv = best[v];
        int pr = kPathNone;
        if (v > 0 && bv > 0) {
            for (int e = s_ptr[v]; e < s_ptr[v + 1]; ++e) {
                const int p = parent_at(e);
                if (p < 0 || p >= v) continue;
                if (best[p] == bv - 1 && p < pr && ok_at(e, p, v)) pr = p;
            }
        }
        pred[v] = pr;
        // end node: longest, then lowest index
        if (bv >= 0) key = max(key, (bv << 10) | (1023 - v));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xFFFFFFFFu, key, o));
    if ((tid & 31) == 0) s_red[tid >> 5] = key;
    if (flags) atomicOr(&s_flags, flags);
    __syncthreads();

    if (tid == 0) {
        for (int w = 1; w < kPathThreads / 32; ++w) key = max(key, s_red[w]);
        const int m = key >> 10;
        int v = 1023 - (key & 1023);
        s_end = v;
        unsigned fl = s_flags;
        if (m + 1 > io.Tcap) fl |= GSD_DEV_TCAP;
        // walk back along the predecessors (cannot break off for a consistent best[])
        for (int len = m; len >= 0; --len) {
            s_path[len] = (short)v;
            if (len == 0) break;
            const int pr = pred[v];
            v = pr == kPathNone ? 0 : pr;
        }
        *io.out_len = m + 1;
        s_m = m;
        if (fl && io.status) atomicOr((unsigned*)io.status, fl);
    }
    __syncthreads();
    const int m = s_m;
    for (int i = tid; i <= io.Tcap; i += kPathThreads) {
        if (i <= m) {
            const int node = s_path[i];
            if (!GSD_IN_BOUNDS(node >= 0 && node < N && i < GSD_MAX_NODES, io.status)) continue;
            if (io.out_nodes && i < io.Tcap) io.out_nodes[i] = node;
            if (i >= 1) io.out_tok[i - 1] = s_tok[node];    // i - 1 < Tcap
        } else if (i < io.Tcap) {
            io.out_tok[i] = -1;
            if (io.out_nodes) io.out_nodes[i] = -1;
        }
    }
    bool end_has_child = false;
    if (kCacheOutcome) {
        int has = 0;
        const int end = s_end;
        for (int v = end + 1 + tid; v < N; v += kPathThreads)
            for (int e = s_ptr[v]; e < s_ptr[v + 1]; ++e) has |= (parent_at(e) == end);
        end_has_child = __syncthreads_or(has) != 0;
    }
    return PathResult{s_m, s_end, end_has_child};
}

// The plain form: a test `step_ok(p, v)` that needs nothing fetched and nothing waited for.
template <bool kCacheOutcome, class StepOk>
__device__ PathResult longest_accepted_path(const PathIo& io, unsigned flags, StepOk step_ok) {
    return longest_accepted_path_ex<kCacheOutcome>(
        io, flags, [&](float, int p, int v) { return step_ok(p, v); }, [](int, int) { return 0.f; }, []() { return 0u; });
}

}  // namespace gsd
