// gsd_draft_expand: one growth step of the draft token graph (Sec. 4: token tree of out-degree
// k; Sec. 4.2: probability pruning and sibling pruning; Sec. 5.2: tau-redundant nodes; Sec. 5.3:
// merge edges to the first occurrence).
//
// Two launches.  Grid (F, B): the CTA of frontier row (b, fi) streams that row of draft logits
// once with 16-byte loads - softmax statistics and every thread's two best (logit, token)
// pairs - lets one warp pick the row's k best among the 512 pairs, and leaves tokens and
// probabilities in scratch (a row where a thread's second pair is picked is redone exactly).
// The second launch (one CTA per sequence, a programmatic dependent of the first) appends the
// children (k per frontier node, in frontier order), applies the two pruning rules, looks for
// an earlier node with the same tau-gram for every new node (first occurrence = lowest id),
// and compacts the new frontier.
#include "gsd_internal.cuh"
#include <math_constants.h>

namespace gsd {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int K = GSD_DRAFT_MAX_K;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// a candidate ranks before another if its logit is larger, or equal with the lower token id
__device__ __forceinline__ bool before(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

struct TopK {
    float v[K];
    int i[K];
};

// insertion into the thread's list (descending).  A thread meets its elements in ascending
// index order, so an equal value never displaces an earlier one.
__device__ __forceinline__ void offer(TopK& t, float x, int idx) {
    if (!(x > t.v[K - 1])) return;
#pragma unroll
    for (int j = K - 1; j >= 0; --j) {
        const bool up = j > 0 && x > t.v[j - 1];     // the slot above also has to move down
        if (up) {
            t.v[j] = t.v[j - 1];
            t.i[j] = t.i[j - 1];
        } else {
            t.v[j] = x;
            t.i[j] = idx;
            break;
        }
    }
}

struct DraftArgs {
    const float* logits;
    const int32_t* frontier;
    const int32_t* frontier_len;
    int32_t* tokens;
    int32_t* tree_parent;
    int32_t* merge_to;
    uint8_t* leaf;
    float* prob;
    int32_t* num_nodes;
    int32_t* new_frontier;
    int32_t* new_frontier_len;
    int32_t* wk_tok;     // [B,F,K]
    float* wk_q;         // [B,F,K]
    int32_t* status;
    int B, F, V, Ncap, k, tau;
    float theta_prob, theta_sib;
};

__device__ void grow_sequence(const DraftArgs& a, int b) {
    __shared__ int s_tok[GSD_MAX_NODES];
    __shared__ int s_par[GSD_MAX_NODES];
    __shared__ unsigned char s_leaf[GSD_MAX_NODES];
    __shared__ __align__(16) unsigned s_key[GSD_MAX_NODES];   // hash of the tau-gram that ends at a node (kNoGram: none)
    __shared__ int s_cnt[kWarps];
    constexpr int kHashBits = 10, kHashSlots = 1 << kHashBits;     // twice the largest node count
    __shared__ unsigned s_hkey[kHashSlots];
    __shared__ int s_hmin[kHashSlots];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int Ncap = a.Ncap, k = a.k;
    int32_t* tok = a.tokens + (size_t)b * Ncap;
    int32_t* par = a.tree_parent + (size_t)b * Ncap;
    int32_t* mrg = a.merge_to + (size_t)b * Ncap;
    uint8_t* leaf = a.leaf + (size_t)b * Ncap;
    float* prob = a.prob + (size_t)b * Ncap;
    unsigned flags = 0;
    int n0 = a.num_nodes[b];
    int fl = a.frontier_len[b];
    if (n0 < 1 || n0 > Ncap || fl < 0 || fl > a.F) {
        // nothing sensible can be appended: leave the graph as it is
        if (tid == 0) {
            a.new_frontier_len[b] = 0;
            if (a.status) atomicOr((unsigned*)a.status, GSD_DEV_BAD_FRONTIER);
        }
        return;
    }
    int want = fl * k;
    if (n0 + want > Ncap) {
        want = Ncap - n0;
        flags |= GSD_DEV_DRAFT_FULL;
    }
    const int n1 = n0 + want;
    // Everything that does not need the row kernel's results comes first - this kernel is its
    // programmatic dependent and is resident while it still runs: the graph as it stands, the
    // parents of the children to come, the tau-gram hashes of the old nodes and their entries in
    // the hash table.
    constexpr int kChildSlots = (GSD_MAX_NODES + kThreads - 1) / kThreads;
    int p_child[kChildSlots];
#pragma unroll
    for (int s = 0; s < kChildSlots; ++s) {
        const int j = tid + s * kThreads;
        int p = 0;
        if (j < want) {
            p = a.frontier[(size_t)b * a.F + j / k];
            if (p < 0 || p >= n0) {
                flags |= GSD_DEV_BAD_FRONTIER;
                p = 0;
            }
        }
        p_child[s] = p;
    }
    for (int v = tid; v < n0; v += kThreads) {
        s_tok[v] = tok[v];
        s_par[v] = par[v];
    }
    constexpr unsigned kNoGram = 0xFFFFFFFFu;
    for (int t = tid; t < kHashSlots; t += kThreads) {
        s_hkey[t] = kNoGram;
        s_hmin[t] = 0x7FFFFFFF;
    }
    __syncthreads();
    // Sec. 5.2 / 5.3: a new node whose last tau tokens along its tree path equal those of an
    // earlier node is redundant; it becomes a leaf that points at the first such node.
    // Every node's tau-gram is reduced to a 32-bit hash; equal hashes are confirmed token by token.
    auto gram_key = [&](int v) -> unsigned {
        unsigned h = 2166136261u;
        int x = v, t = 0;
        for (; t < a.tau && x >= 0; ++t) {
            h = (h ^ (unsigned)s_tok[x]) * 16777619u;
            h ^= h >> 15;
            x = s_par[x];
        }
        return (t == a.tau) ? (h == kNoGram ? 0u : h) : kNoGram;
    };
    // first occurrences through a hash table in shared memory: every node with a tau-gram enters
    // its id under its hash (open addressing; the slot keeps the lowest id), so a new node finds
    // the lowest earlier node with its hash in one probe sequence instead of a scan over all
    // earlier nodes.  Equal hashes are confirmed token by token; if the lowest id under the hash
    // is a different gram (a collision of the 32-bit hash) the node falls back to the scan.
    auto enter = [&](int v) {
        const unsigned kv = gram_key(v);
        s_key[v] = kv;
        if (kv == kNoGram) return;
        unsigned slot = (kv * 2654435761u) >> (32 - kHashBits);
        for (int probe = 0; probe < kHashSlots; ++probe) {
            const unsigned prev = atomicCAS(&s_hkey[slot], kNoGram, kv);
            if (prev == kNoGram || prev == kv) {
                atomicMin(&s_hmin[slot], v);
                break;
            }
            slot = (slot + 1) & (kHashSlots - 1);
        }
    };
    for (int v = tid; v < n0; v += kThreads) enter(v);

    // the children: k per frontier node, in frontier order, best first
    asm volatile("griddepcontrol.wait;" ::: "memory");
#pragma unroll
    for (int s = 0; s < kChildSlots; ++s) {
        const int j = tid + s * kThreads;
        if (j >= want) continue;
        const int fi = j / k, i = j % k, c = n0 + j;
        const size_t w = ((size_t)b * a.F + fi) * K;
        if (!GSD_IN_BOUNDS(c < Ncap && fi < a.F && i < K, a.status)) continue;
        const float q = a.wk_q[w + i], qmax = a.wk_q[w];
        s_tok[c] = a.wk_tok[w + i];
        s_par[c] = p_child[s];
        // Sec. 4.2: below the probability threshold, or too far below the best sibling
        s_leaf[c] = (q < a.theta_prob) || (q < a.theta_sib * qmax);
        prob[c] = q;
    }
    __syncthreads();
    for (int v = n0 + tid; v < n1; v += kThreads) enter(v);
    auto same_gram = [&](int x, int y) -> bool {
        for (int t = 0; t < a.tau; ++t) {
            if (x < 0 || y < 0 || s_tok[x] != s_tok[y]) return false;
            x = s_par[x];
            y = s_par[y];
        }
        return true;
    };
    __syncthreads();
    for (int j = tid; j < want; j += kThreads) {
        const int c = n0 + j;
        const unsigned kc = s_key[c];
        int first = -1;
        if (kc != kNoGram) {
            unsigned slot = (kc * 2654435761u) >> (32 - kHashBits);
            int lowest = c;
            for (int probe = 0; probe < kHashSlots; ++probe) {
                const unsigned k = s_hkey[slot];
                if (k == kc) { lowest = s_hmin[slot]; break; }
                if (k == kNoGram) break;                       // (cannot happen: c itself is in the table)
                slot = (slot + 1) & (kHashSlots - 1);
            }
            if (lowest < c) {
                if (same_gram(c, lowest)) {
                    first = lowest;
                } else {
                    // another gram with the same hash sits below: look at every earlier node
                    for (int e = 0; e < c && first < 0; ++e)
                        if (s_key[e] == kc && same_gram(c, e)) first = e;
                }
            }
        }
        if (first >= 0) s_leaf[c] = 1;
        tok[c] = s_tok[c];
        par[c] = s_par[c];
        mrg[c] = first;
        leaf[c] = s_leaf[c];
    }
    __syncthreads();
    // the new frontier: the new nodes that are not leaves, in id order
    int32_t* nf = a.new_frontier + (size_t)b * a.F * k;
    int base = 0;
    for (int j0 = 0; j0 < want; j0 += kThreads) {
        const int j = j0 + tid;
        const bool keep = j < want && !s_leaf[n0 + j];
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, keep);
        if (lane == 0) s_cnt[warp] = __popc(bal);
        __syncthreads();
        int off = base;
        for (int w = 0; w < warp; ++w) off += s_cnt[w];
        if (keep && GSD_IN_BOUNDS(off + __popc(bal & ((1u << lane) - 1u)) < a.F * k, a.status))
            nf[off + __popc(bal & ((1u << lane) - 1u))] = n0 + j;
        for (int w = 0; w < kWarps; ++w) base += s_cnt[w];
        __syncthreads();
    }
    if (tid == 0) {
        a.new_frontier_len[b] = base;
        a.num_nodes[b] = n1;
    }
    if (flags && a.status) atomicOr((unsigned*)a.status, flags);
}

// Block-wide pick of the best remaining (value, index) pair, ranked by `before`; every thread
// passes its own proposal and gets the winner (and the proposing thread) back.
__device__ __forceinline__ void block_best(float& v, int& i, int& owner, float* s_rv, int* s_ri, int* s_rt) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v2 = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        const int i2 = __shfl_xor_sync(0xFFFFFFFFu, i, o), t2 = __shfl_xor_sync(0xFFFFFFFFu, owner, o);
        if (before(v2, i2, v, i)) { v = v2; i = i2; owner = t2; }
    }
    if (lane == 0) { s_rv[warp] = v; s_ri[warp] = i; s_rt[warp] = owner; }
    __syncthreads();
    v = s_rv[0]; i = s_ri[0]; owner = s_rt[0];
    for (int q = 1; q < kWarps; ++q)
        if (before(s_rv[q], s_ri[q], v, i)) { v = s_rv[q]; i = s_ri[q]; owner = s_rt[q]; }
    __syncthreads();
}

// The k best tokens of one row of logits and their probabilities, in one pass over the row.
// Every thread streams its strided share (16-byte loads, kBatch in flight) and keeps the running
// (maximum, sum of exponentials) pair, the best (logit, token) pair it has met and the VALUE of
// its second best entry - all without a branch, so that no lane of a warp waits for another's
// rare update.  The 256 best pairs are picked over in two stages, both with shuffles only (ranked
// by logit, ties to the lower token id): every warp picks the k best of its 32 pairs, then one
// warp picks the k best of those 8 k.  That is the exact answer unless some thread's second best
// entry ranks at or before the k-th pick - then an entry that no thread offered could belong
// to the k best (for a random row: about one row in fifty).  Such a row is read once more (from
// L2): the k-th pick bounds the k-th best entry from below, the entries at or before it form a
// short list, and the pick is repeated over the list.  Only a list longer than 512 (long runs
// of equal logits) takes the slow exact way: every thread keeps the K best pairs it meets and
// the block merges the 256 lists.
constexpr int kBatch = 8;     // 16-byte loads a thread keeps in flight while it streams a row
struct Best {
    float v1, v2;   // best and second best logit of the thread's share (v2: value only)
    int i1;         // token of the best
};
__device__ __forceinline__ void offer_best(Best& t, float x, int idx) {
    // a thread meets its entries in ascending token order: an equal logit never displaces an earlier one
    const bool up = x > t.v1;
    t.v2 = fmaxf(t.v2, up ? t.v1 : x);
    t.i1 = up ? idx : t.i1;
    t.v1 = up ? x : t.v1;
}
// The best of the pairs the 32 lanes hold (ranked by `before`), and the lane that held it.
__device__ __forceinline__ void warp_best(float& v, int& i, int& src) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v2 = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        const int i2 = __shfl_xor_sync(0xFFFFFFFFu, i, o), s2 = __shfl_xor_sync(0xFFFFFFFFu, src, o);
        if (before(v2, i2, v, i)) { v = v2; i = i2; src = s2; }
    }
}

// One warp picks the k best of `count` <= 512 (logit, token) pairs in shared memory with
// shuffles only and writes tokens and probabilities to the row's scratch entries.  Returns (to
// every lane) bit 0: a pair in an odd slot was picked; bit 1: fewer than k pairs above -inf;
// the k-th pick is left in (*last_v, *last_i).
__device__ __forceinline__ int warp_pick_k(const float* s_cv, const int* s_ci, int count, int k, float rm, float rs,
                                           int32_t* wk_tok, float* wk_q, float* last_v, int* last_i) {
    const int lane = threadIdx.x & 31;
    float cv[16];
    int ci[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const bool in = lane + 32 * j < count;
        cv[j] = in ? s_cv[lane + 32 * j] : -CUDART_INF_F;
        ci[j] = in ? s_ci[lane + 32 * j] : 0x7FFFFFFF;
    }
    int result = 0;
    float v = -CUDART_INF_F;
    int i = 0x7FFFFFFF;
    for (int r = 0; r < k; ++r) {
        v = -CUDART_INF_F;
        i = 0x7FFFFFFF;
        int slot = -1;
#pragma unroll
        for (int j = 0; j < 16; ++j)
            if (before(cv[j], ci[j], v, i)) { v = cv[j]; i = ci[j]; slot = lane + 32 * j; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float v2 = __shfl_xor_sync(0xFFFFFFFFu, v, o);
            const int i2 = __shfl_xor_sync(0xFFFFFFFFu, i, o), t2 = __shfl_xor_sync(0xFFFFFFFFu, slot, o);
            if (before(v2, i2, v, i)) { v = v2; i = i2; slot = t2; }
        }
        // pairs at -inf are never taken (slot stays -1 when nothing above -inf is left)
        if (slot >= 0) {
            if (slot & 1) result |= 1;
#pragma unroll
            for (int j = 0; j < 16; ++j)
                if (slot == lane + 32 * j) { cv[j] = -CUDART_INF_F; ci[j] = 0x7FFFFFFF; }
        } else {
            result |= 2;
        }
        if (lane == 0) {
            wk_tok[r] = slot < 0 ? -1 : i;
            wk_q[r] = slot < 0 ? 0.f : ex2((v - rm) * kLog2e) / rs;
        }
    }
    *last_v = v;
    *last_i = i;
    return result;
}

template <bool kVec>
__global__ void __launch_bounds__(kThreads, 4) draft_expand_kernel(DraftArgs a) {
    __shared__ float s_cv[2 * kThreads];
    __shared__ int s_ci[2 * kThreads];
    __shared__ float s_rv[kWarps];
    __shared__ int s_ri[kWarps], s_rt[kWarps];
    __shared__ float s_m[kWarps], s_s[kWarps], s_v2[kWarps];
    __shared__ int s_redo, s_count, s_ti;
    __shared__ float s_tv;
    // the per-sequence pass (a programmatic dependent launch) may become resident as CTAs retire
    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int fi = blockIdx.x, b = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = a.V;
    const int fl = a.frontier_len[b];
    if (fi >= fl || fl > a.F) return;
    const float* x = a.logits + ((size_t)b * a.F + fi) * V;
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const int nvec = V >> 2;
    float m = -CUDART_INF_F, s = 0.f;        // running maximum and sum
    Best best{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
    auto take = [&](float val, int idx) {
        offer_best(best, val, idx);
        if (val > m) {
            s = s * ex2((m - val) * kLog2e) + 1.f;
            m = val;
        } else if (val > -CUDART_INF_F) {
            s += ex2((val - m) * kLog2e);
        } else if (val != val) {
            s = val;    // NaN poisons the sum and is reported below
        }
    };
    if (kVec) {
        const float4 none = make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
        for (int i = tid; i < nvec; i += kBatch * kThreads) {
            float4 r[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) r[k] = i + k * kThreads < nvec ? __ldcs(x4 + i + k * kThreads) : none;
            float g = m;
            float nan_probe = 0.f;
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const float g4 = fmaxf(fmaxf(r[k].x, r[k].y), fmaxf(r[k].z, r[k].w));
                g = fmaxf(g, g4);
                nan_probe += (r[k].x + r[k].y) + (r[k].z + r[k].w);     // NaN if any entry is NaN (or +inf and -inf meet)
                const int e = (i + k * kThreads) * 4;
                offer_best(best, r[k].x, e); offer_best(best, r[k].y, e + 1);
                offer_best(best, r[k].z, e + 2); offer_best(best, r[k].w, e + 3);
            }
            if (nan_probe != nan_probe) {
                // rare: find out entry by entry (a NaN poisons the sum; -inf next to +inf does not)
#pragma unroll
                for (int k = 0; k < kBatch; ++k) {
                    const float q[4] = {r[k].x, r[k].y, r[k].z, r[k].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (q[j] != q[j]) s = q[j];
                }
            }
            if (g == -CUDART_INF_F) continue;      // nothing finite yet
            // one rescale per batch
            const float kk = -g * kLog2e;
            float acc = s * ex2(fmaf(m, kLog2e, kk));
#pragma unroll
            for (int k = 0; k < kBatch; ++k)
                acc += (ex2(fmaf(r[k].x, kLog2e, kk)) + ex2(fmaf(r[k].y, kLog2e, kk))) + (ex2(fmaf(r[k].z, kLog2e, kk)) + ex2(fmaf(r[k].w, kLog2e, kk)));
            s = acc;
            m = g;
        }
    } else {
        for (int i = tid; i < V; i += kThreads) take(__ldcs(x + i), i);
    }
    // stage 1: every warp picks the k best of its 32 pairs; lane r keeps the r-th pick
    {
        float cv = best.v1, pv = -CUDART_INF_F;
        int ci = best.i1, pi = 0x7FFFFFFF;
        for (int r = 0; r < a.k; ++r) {
            float v = cv;
            int i = ci, src = lane;
            warp_best(v, i, src);
            if (lane == r) { pv = v; pi = i; }
            if (src == lane) { cv = -CUDART_INF_F; ci = 0x7FFFFFFF; }      // (a pair at -inf is never taken: its token is none)
        }
        if (lane < a.k) { s_cv[warp * K + lane] = pv; s_ci[warp * K + lane] = pi; }
        float v2 = best.v2;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v2 = fmaxf(v2, __shfl_xor_sync(0xFFFFFFFFu, v2, o));
        if (lane == 0) s_v2[warp] = v2;
    }
    // (maximum, sum) of the row
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xFFFFFFFFu, m, o), s2 = __shfl_xor_sync(0xFFFFFFFFu, s, o);
        const float mm = fmaxf(m, m2);
        s = (mm == -CUDART_INF_F) ? ((s != s || s2 != s2) ? CUDART_NAN_F : 0.f)
                                  : s * ex2((m - mm) * kLog2e) + s2 * ex2((m2 - mm) * kLog2e);
        m = mm;
    }
    if (lane == 0) { s_m[warp] = m; s_s[warp] = s; }
    if (tid == 0) s_redo = 0;
    __syncthreads();
    float rm = -CUDART_INF_F, rs = 0.f;
    const size_t w = ((size_t)b * a.F + fi) * K;
    if (warp == 0) {
        for (int q = 0; q < kWarps; ++q) {
            const float mm = fmaxf(rm, s_m[q]);
            rs = (mm == -CUDART_INF_F) ? ((rs != rs || s_s[q] != s_s[q]) ? CUDART_NAN_F : 0.f)
                                       : rs * ex2((rm - mm) * kLog2e) + s_s[q] * ex2((s_m[q] - mm) * kLog2e);
            rm = mm;
        }
        if (lane == 0 && (!(rs > 0.f) || rm == CUDART_INF_F) && a.status) atomicOr((unsigned*)a.status, GSD_DEV_BAD_LOGITS);
        // stage 2: the k best of the 8 k picks (two per lane at most)
        const int n = kWarps * a.k;
        float c0 = -CUDART_INF_F, c1 = -CUDART_INF_F;
        int j0 = 0x7FFFFFFF, j1 = 0x7FFFFFFF;
        if (lane < n) { c0 = s_cv[(lane / a.k) * K + lane % a.k]; j0 = s_ci[(lane / a.k) * K + lane % a.k]; }
        if (lane + 32 < n) { c1 = s_cv[((lane + 32) / a.k) * K + (lane + 32) % a.k]; j1 = s_ci[((lane + 32) / a.k) * K + (lane + 32) % a.k]; }
        float tv = -CUDART_INF_F;
        int ti = 0x7FFFFFFF;
        bool short_row = false;
        for (int r = 0; r < a.k; ++r) {
            const bool second = before(c1, j1, c0, j0);
            float v = second ? c1 : c0;
            int i = second ? j1 : j0, src = lane;
            warp_best(v, i, src);
            if (src == lane) {
                if (second) { c1 = -CUDART_INF_F; j1 = 0x7FFFFFFF; } else { c0 = -CUDART_INF_F; j0 = 0x7FFFFFFF; }
            }
            const bool none = i == 0x7FFFFFFF;
            short_row |= none;
            if (lane == 0) {
                a.wk_tok[w + r] = none ? -1 : i;
                a.wk_q[w + r] = none ? 0.f : ex2((v - rm) * kLog2e) / rs;
            }
            tv = v;
            ti = i;
        }
        // an entry that no thread offered can rank at or before the k-th pick only if some
        // thread's second best does
        float v2 = lane < kWarps ? s_v2[lane] : -CUDART_INF_F;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v2 = fmaxf(v2, __shfl_xor_sync(0xFFFFFFFFu, v2, o));
        const bool redo = v2 > -CUDART_INF_F && v2 >= tv;
        if (lane == 0) {
            s_redo = redo ? 1 : 0;
            s_tv = tv;
            s_ti = ti;
            s_count = 0;
            // (a row that goes through the second pass finds out there whether it is short of k entries)
            if (short_row && !redo && a.status) atomicOr((unsigned*)a.status, GSD_DEV_BAD_LOGITS);
        }
    }
    __syncthreads();
    if (!s_redo) return;
    // Second pass (about one random row in fifty): the k-th pick is a lower bound on the row's
    // k-th best entry, so everything that ranks at or before it is collected from the row (now
    // in L2) and the pick is repeated over that list.
    const float tv = s_tv;
    const int ti = s_ti;
    __syncthreads();                        // the pairs have been read: the list takes their place
    auto consider = [&](float val, int idx) {
        if (val > tv || (val == tv && idx <= ti)) {
            const int slot = atomicAdd(&s_count, 1);
            if (slot < 2 * kThreads) { s_cv[slot] = val; s_ci[slot] = idx; }
        }
    };
    if (kVec) {
        const float4 none = make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
        for (int i = tid; i < nvec; i += 8 * kThreads) {
            float4 r[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) r[k] = i + k * kThreads < nvec ? x4[i + k * kThreads] : none;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int e = (i + k * kThreads) * 4;
                if (fmaxf(fmaxf(r[k].x, r[k].y), fmaxf(r[k].z, r[k].w)) >= tv) {
                    consider(r[k].x, e); consider(r[k].y, e + 1); consider(r[k].z, e + 2); consider(r[k].w, e + 3);
                }
            }
        }
    } else {
        for (int i = tid; i < V; i += kThreads) consider(x[i], i);
    }
    __syncthreads();
    const int count = s_count;
    if (count <= 2 * kThreads) {
        if (warp == 0) {
            float lv;
            int li;
            const int res = warp_pick_k(s_cv, s_ci, count, a.k, rm, rs, a.wk_tok + w, a.wk_q + w, &lv, &li);
            if (lane == 0 && (res & 2) && a.status) atomicOr((unsigned*)a.status, GSD_DEV_BAD_LOGITS);
        }
        return;
    }
    {
        // more than 512 entries rank before the bound (long runs of equal logits in one thread's
        // share): per-thread lists of the K best pairs, merged by the block
        TopK t;
#pragma unroll
        for (int j = 0; j < K; ++j) {
            t.v[j] = -CUDART_INF_F;
            t.i[j] = 0x7FFFFFFF;
        }
        if (kVec) {
            for (int i = tid; i < nvec; i += kThreads) {
                const float4 r = x4[i];
                offer(t, r.x, 4 * i); offer(t, r.y, 4 * i + 1); offer(t, r.z, 4 * i + 2); offer(t, r.w, 4 * i + 3);
            }
        } else {
            for (int i = tid; i < V; i += kThreads) offer(t, x[i], i);
        }
        int head = 0;
        for (int r = 0; r < a.k; ++r) {
            float v = -CUDART_INF_F;
            int i = 0x7FFFFFFF;
#pragma unroll
            for (int j = 0; j < K; ++j)
                if (j == head) { v = t.v[j]; i = t.i[j]; }
            int owner = tid;
            block_best(v, i, owner, s_rv, s_ri, s_rt);
            if (owner == tid && i != 0x7FFFFFFF) ++head;
            if (tid == 0) {
                if (i == 0x7FFFFFFF && a.status) atomicOr((unsigned*)a.status, GSD_DEV_BAD_LOGITS);   // fewer than k entries above -inf
                a.wk_tok[w + r] = i == 0x7FFFFFFF ? -1 : i;
                a.wk_q[w + r] = v == -CUDART_INF_F ? 0.f : ex2((v - rm) * kLog2e) / rs;
            }
        }
    }
}

// Second launch: one CTA per sequence appends the children and updates the graph once every
// row's result of the first launch is visible.
__global__ void __launch_bounds__(kThreads) draft_grow_kernel(DraftArgs a) {
    grow_sequence(a, blockIdx.x);        // (waits for the first launch inside, as late as it can)
}

}  // namespace
}  // namespace gsd

extern "C" size_t gsd_draft_expand_workspace_bytes(const gsd_draft_params* p) {
    if (!p || p->B < 1 || p->F < 1) return 0;
    return gsd::align_up((size_t)p->B * p->F * GSD_DRAFT_MAX_K * 8, 256);
}

extern "C" int gsd_draft_expand(const float* logits, const int32_t* frontier, const int32_t* frontier_len,
                                int32_t* tokens, int32_t* tree_parent, int32_t* merge_to, uint8_t* leaf,
                                float* prob, int32_t* num_nodes, int32_t* new_frontier,
                                int32_t* new_frontier_len, const gsd_draft_params* p, void* workspace,
                                size_t workspace_bytes, int32_t* status, void* stream) {
    using namespace gsd;
    if (!p || !logits || !frontier || !frontier_len || !tokens || !tree_parent || !merge_to || !leaf ||
        !prob || !num_nodes || !new_frontier || !new_frontier_len)
        return GSD_ERR_NULL_POINTER;
    if (p->B < 1 || p->B > 65535 || p->F < 1 || p->V < 1 || p->Ncap < 1 || p->Ncap > GSD_MAX_NODES ||
        p->k < 1 || p->k > GSD_DRAFT_MAX_K || p->k > p->V || p->tau < 1 || p->tau > GSD_MAX_NODES)
        return GSD_ERR_BAD_SHAPE;
    if (((uintptr_t)logits & 3u) != 0) return GSD_ERR_MISALIGNED;
    const size_t need = gsd_draft_expand_workspace_bytes(p);
    if (!workspace || workspace_bytes < need) return GSD_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 7u) != 0) return GSD_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    DraftArgs a;
    a.logits = logits; a.frontier = frontier; a.frontier_len = frontier_len;
    a.tokens = tokens; a.tree_parent = tree_parent; a.merge_to = merge_to; a.leaf = leaf; a.prob = prob;
    a.num_nodes = num_nodes; a.new_frontier = new_frontier; a.new_frontier_len = new_frontier_len;
    const size_t rows = (size_t)p->B * p->F * GSD_DRAFT_MAX_K;
    a.wk_tok = (int32_t*)workspace;
    a.wk_q = (float*)((char*)workspace + rows * 4);
    a.status = status;
    a.B = p->B; a.F = p->F; a.V = p->V; a.Ncap = p->Ncap; a.k = p->k; a.tau = p->tau;
    a.theta_prob = p->theta_prob; a.theta_sib = p->theta_sib;
    // every scratch entry is written before it is read: nothing has to start at zero
    const bool vec = (p->V % 4 == 0) && (((uintptr_t)logits & 15u) == 0);
    dim3 grid((unsigned)p->F, (unsigned)p->B);
    if (vec) draft_expand_kernel<true><<<grid, kThreads, 0, st>>>(a);
    else draft_expand_kernel<false><<<grid, kThreads, 0, st>>>(a);
    GSD_CUDA_TRY(cudaGetLastError());
    cudaLaunchAttribute attr[1];
    dependent_launch_attr(attr);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p->B);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    GSD_CUDA_TRY(cudaLaunchKernelEx(&cfg, draft_grow_kernel, a));
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}
