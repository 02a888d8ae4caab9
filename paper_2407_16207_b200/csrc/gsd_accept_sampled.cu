// gsd_accept_sampled: non-deterministic verification of the draft token graph (Sec. 3: a
// drafted token is accepted with probability min(1, p/q), the first rejection ends the
// hypothesis and the target model regenerates that token; Sec. 6.4: the same on the graph).
// The random numbers are inputs.  A step parent -> v of the graph is accepted iff
//     u_accept[v] * draft_q[v] < softmax(logits[parent])[token of v];
// the hypothesis is the longest root path of accepted steps (ties as in gsd_accept), and the
// regenerated token is drawn by inverting a cumulative distribution in index order with
// u_sample: that of the residual max(0, P - Q) at the end node (P the target's, Q the draft
// model's distribution there) when drafted continuations of the end node were rejected, that of
// P itself when the end node is a leaf of the graph or no draft logits are given.
//
// Two launches.  Grid (slices, B*N): each CTA streams one slice of one logits row with 16-byte
// loads; each of its warps owns a contiguous eighth of the slice and keeps a running
// (maximum, sum of exponentials) pair, which it leaves in scratch.  The second launch (one CTA
// per sequence, a programmatic dependent of the first, so it is resident when the stream ends)
// combines the pairs per node, tests the steps, runs the level-synchronous longest-path
// relaxation, walks back, and finds the regenerated token: range sums (for P those in scratch;
// for the residual eight range sums formed on the spot from the two rows of the end node) give
// the range of the crossing, a block-wide scan over that range gives the index.
#include "gsd_internal.cuh"
#include "gsd_path.cuh"
#include <math_constants.h>

namespace gsd {
namespace {

constexpr int kThreads = kPathThreads;
constexpr int kNone = 0x7FFFFFFF;
constexpr int kMaxSlices = 16;
constexpr int kWarps = kThreads / 32;   // each warp of a CTA sums a contiguous eighth of the CTA's slice
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kResidualFloor = 1e-6f;   // a residual mass at or below this is rounding noise

// (maximum, sum of 2^((x - maximum) * log2 e)) of a set of logits; the empty set is (-inf, 0)
struct Ms {
    float m, s;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ Ms combine(Ms a, Ms b) {
    const float m = fmaxf(a.m, b.m);
    if (m == -CUDART_INF_F) return Ms{m, 0.f};
    return Ms{m, a.s * ex2((a.m - m) * kLog2e) + b.s * ex2((b.m - m) * kLog2e)};
}

// sixteen values at once: one rescale of the running sum per group
__device__ __forceinline__ void take16(Ms& r, const float4& a, const float4& b, const float4& c, const float4& d) {
    const float m4 = fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w)));
    const float m8 = fmaxf(fmaxf(fmaxf(c.x, c.y), fmaxf(c.z, c.w)), fmaxf(fmaxf(d.x, d.y), fmaxf(d.z, d.w)));
    const float m = fmaxf(r.m, fmaxf(m4, m8));
    if (m == -CUDART_INF_F) return;
    const float k = -m * kLog2e;
    float s = r.s * ex2(fmaf(r.m, kLog2e, k));
    s += ex2(fmaf(a.x, kLog2e, k)) + ex2(fmaf(a.y, kLog2e, k)) + ex2(fmaf(a.z, kLog2e, k)) + ex2(fmaf(a.w, kLog2e, k));
    s += ex2(fmaf(b.x, kLog2e, k)) + ex2(fmaf(b.y, kLog2e, k)) + ex2(fmaf(b.z, kLog2e, k)) + ex2(fmaf(b.w, kLog2e, k));
    s += ex2(fmaf(c.x, kLog2e, k)) + ex2(fmaf(c.y, kLog2e, k)) + ex2(fmaf(c.z, kLog2e, k)) + ex2(fmaf(c.w, kLog2e, k));
    s += ex2(fmaf(d.x, kLog2e, k)) + ex2(fmaf(d.y, kLog2e, k)) + ex2(fmaf(d.z, kLog2e, k)) + ex2(fmaf(d.w, kLog2e, k));
    r.m = m;
    r.s = s;
}

__device__ __forceinline__ void take1(Ms& r, float x) {
    r = combine(r, Ms{x, x == -CUDART_INF_F ? 0.f : 1.f});
}

// The row is cut into slices (one CTA each) and every slice into kWarps contiguous ranges (one
// warp each); in units of float4 when the row is read that way.  Range r = slice * kWarps + warp.
__device__ __forceinline__ void range_of(int V, int slices, int vec, int r, int& lo, int& hi) {
    const int unit = vec ? 4 : 1, n = vec ? (V >> 2) : V;
    const int per = (n + slices - 1) / slices;
    const int slice = r / kWarps, warp = r % kWarps;
    const int v0 = min(slice * per, n), v1 = min(v0 + per, n);
    const int wlen = (v1 - v0 + kWarps - 1) / kWarps;
    const int a0 = min(v0 + warp * wlen, v1), a1 = min(a0 + wlen, v1);
    lo = a0 * unit;
    hi = a1 * unit;
}

struct SampledArgs {
    const float* logits;
    const float* dlogits;  // draft-model logits [B,N,V] or nullptr (then no residual is formed)
    const int32_t* tok;
    const int32_t* pptr;
    const int32_t* pidx;
    const float* q;
    const float* u;
    const float* us;
    int32_t* out_tok;
    int32_t* out_len;
    int32_t* out_nodes;
    float2* part;     // [B*N][slices][kWarps] (maximum, sum) of contiguous ranges of the row, in order
    int32_t* status;
    int B, N, V, Ecap, Tcap, slices;
    int vec;          // rows are read as float4 (decides where the slices of a row begin)
    int dvec;         // the rows of the draft logits can be read as float4 too
};

__device__ void finish_sequence(const SampledArgs& a, int b) {
    __shared__ float s_mx[GSD_MAX_NODES];
    __shared__ float s_sum[GSD_MAX_NODES];
    __shared__ float s_uq[GSD_MAX_NODES];
    __shared__ int s_red[kThreads / 32];
    __shared__ float s_scan[kThreads / 32];
    __shared__ float s_rm[kThreads / 32];
    __shared__ float s_rsum[kMaxSlices * kWarps];
    __shared__ int s_pick;
    const int N = a.N, V = a.V, tid = threadIdx.x;
    const int32_t* tok = a.tok + (size_t)b * N;
    const float* lg = a.logits + (size_t)b * N * V;
    const float* q = a.q + (size_t)b * N;
    const float* u = a.u + (size_t)b * N;
    // Softmax statistics of every node from the pairs of the first launch, and the left sides
    // of the step tests.  This is the first thing that needs the first launch's results: the path
    // routine calls it after the graph and one logit per step have been fetched, so those two
    // trips to memory are over when the first launch ends.
    auto combine_pairs = [&]() -> unsigned {
        unsigned flags = 0;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int v = tid; v < N; v += kThreads) {
            // the pairs were written by other CTAs: read them past L1
            Ms r{-CUDART_INF_F, 0.f};
            const float4* pp = reinterpret_cast<const float4*>(a.part + ((size_t)b * N + v) * a.slices * kWarps);
            for (int k = 0; k < a.slices * (kWarps / 2); k += 4) {     // eight pairs (64 bytes) per round, loaded at once
                float4 t[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) t[i] = __ldcg(pp + k + i);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    r = combine(r, Ms{t[i].x, t[i].y});
                    r = combine(r, Ms{t[i].z, t[i].w});
                }
            }
            s_mx[v] = r.m;
            s_sum[v] = r.s;
            s_uq[v] = u[v] * q[v];       // the left side of the step test, fetched beside the pairs
            if (!(r.s > 0.f) || r.m == CUDART_INF_F) flags |= GSD_DEV_BAD_LOGITS;   // no finite entry, +inf or NaN
        }
        return flags;
    };
    PathIo io;
    io.tok = tok;
    io.pptr = a.pptr + (size_t)b * (N + 1);
    io.pidx = a.pidx + (size_t)b * a.Ecap;
    io.out_tok = a.out_tok + (size_t)b * a.Tcap;
    io.out_nodes = a.out_nodes ? a.out_nodes + (size_t)b * a.Tcap : nullptr;
    io.out_len = a.out_len + b;
    io.status = a.status;
    io.N = N; io.V = V; io.Ecap = a.Ecap; io.Tcap = a.Tcap;
    // the test of one step: the target's probability of v's token under its parent p (one
    // logit gathered from global memory) against u q
    const PathResult res = longest_accepted_path_ex<true>(
        io, 0u,
        [&](float logit, int p, int v) { return s_uq[v] < ex2((logit - s_mx[p]) * kLog2e) / s_sum[p]; },
        [&](int p, int v) -> float {
            if (!GSD_IN_BOUNDS(p >= 0 && p < N && tok[v] >= 0 && tok[v] < V, a.status)) return -CUDART_INF_F;
            return lg[(size_t)p * V + tok[v]];
        },
        combine_pairs);
    const int s_m = res.edges, s_end = res.end;
    int32_t* out_tok = io.out_tok;

    // The regenerated token: weights w_j over the vocabulary at the end node, then the smallest
    // t whose cumulative weight exceeds u * (total weight).  First the contiguous range of the
    // row that holds the crossing is found from range sums, then the whole block splits that
    // range into 256 contiguous pieces, scans the piece sums, and the thread whose piece holds
    // the crossing walks it.
    const float* x = lg + (size_t)s_end * V;
    const float mx = s_mx[s_end];
    const int lane = tid & 31, warp = tid >> 5;

    // Residual of the sampling scheme: when drafted continuations of the end node were rejected
    // (it has a child in the graph) the weights are max(0, P_j - Q_j), Q the draft model's
    // distribution at that node.  Its range sums are formed here: each warp takes a contiguous
    // eighth of the row with coalesced loads.
    bool residual = false;
    float q_m = 0.f, inv_sp = 0.f, inv_sq = 0.f, res_total = 0.f;
    const float* y = nullptr;
    // both rows readable as float4 (decides where the residual's ranges begin)
    const bool rvec = a.vec && a.dvec;
    const int runit = rvec ? 4 : 1, rn = rvec ? (V >> 2) : V;
    const int rper = (rn + kWarps - 1) / kWarps;
    if (a.dlogits && res.end_has_child) {
        y = a.dlogits + ((size_t)b * N + s_end) * V;
        // softmax statistics of the draft row: the row comes from DRAM, so every thread keeps
        // sixteen 16-byte loads in flight (a 32000-entry row is two trips to memory)
        Ms r{-CUDART_INF_F, 0.f};
        if (a.dvec) {
            const float4* y4 = reinterpret_cast<const float4*>(y);
            const int n4 = V >> 2;
            const float4 none = make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
            for (int i = tid; i < n4; i += 16 * kThreads) {
                float4 t[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) t[k] = i + k * kThreads < n4 ? __ldg(y4 + i + k * kThreads) : none;
#pragma unroll
                for (int k = 0; k < 16; k += 4) take16(r, t[k], t[k + 1], t[k + 2], t[k + 3]);
            }
        } else {
            for (int j = tid; j < V; j += kThreads) take1(r, __ldg(y + j));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            Ms t;
            t.m = __shfl_xor_sync(0xFFFFFFFFu, r.m, o);
            t.s = __shfl_xor_sync(0xFFFFFFFFu, r.s, o);
            r = combine(r, t);
        }
        if (lane == 0) { s_rm[warp] = r.m; s_scan[warp] = r.s; }
        __syncthreads();
        r = Ms{-CUDART_INF_F, 0.f};
        for (int w = 0; w < kWarps; ++w) r = combine(r, Ms{s_rm[w], s_scan[w]});
        __syncthreads();
        if (!(r.s > 0.f) || r.m == CUDART_INF_F) {
            if (tid == 0 && a.status) atomicOr((unsigned*)a.status, GSD_DEV_BAD_LOGITS);
        } else {
            q_m = r.m;
            inv_sp = 1.f / s_sum[s_end];
            inv_sq = 1.f / r.s;
            auto res1 = [&](float xv, float yv) -> float {
                return fmaxf(ex2((xv - mx) * kLog2e) * inv_sp - ex2((yv - q_m) * kLog2e) * inv_sq, 0.f);
            };
            // range sums of the residual: warp w takes the w-th eighth of the row
            const int w0 = min(warp * rper, rn), w1 = min(w0 + rper, rn);
            float part = 0.f;
            if (rvec) {
                const float4* x4 = reinterpret_cast<const float4*>(x);
                const float4* y4 = reinterpret_cast<const float4*>(y);
                const float4 none = make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
                for (int i = w0 + lane; i < w1; i += 8 * 32) {
                    float4 xv[8], yv[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const bool in = i + k * 32 < w1;
                        xv[k] = in ? __ldg(x4 + i + k * 32) : none;
                        yv[k] = in ? __ldg(y4 + i + k * 32) : none;
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        part += (res1(xv[k].x, yv[k].x) + res1(xv[k].y, yv[k].y)) + (res1(xv[k].z, yv[k].z) + res1(xv[k].w, yv[k].w));
                }
            } else {
                for (int j = w0 + lane; j < w1; j += 32) part += res1(x[j], y[j]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
            if (lane == 0) s_scan[warp] = part;
            __syncthreads();
            for (int w = 0; w < kWarps; ++w) res_total += s_scan[w];
            // a residual without mass (the two distributions agree to rounding) leaves P
            residual = res_total > kResidualFloor;
        }
    }
    // weight of one entry from its two logits (-inf stands for "past the end": weight 0)
    auto weight = [&](float xv, float yv) -> float {
        const float e = ex2((xv - mx) * kLog2e);
        return residual ? fmaxf(e * inv_sp - ex2((yv - q_m) * kLog2e) * inv_sq, 0.f) : e;
    };
    // sixteen consecutive entries of a row, all loads issued before any is used
    auto load16 = [&](const float* row, bool vec16, int j, int jend, float (&v)[16]) {
        if (vec16 && (j & 3) == 0 && j + 16 <= jend) {
            const float4* r4 = reinterpret_cast<const float4*>(row + j);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float4 t = r4[k];
                v[4 * k] = t.x; v[4 * k + 1] = t.y; v[4 * k + 2] = t.z; v[4 * k + 3] = t.w;
            }
        } else {
#pragma unroll
            for (int k = 0; k < 16; ++k) v[k] = j + k < jend ? row[j + k] : -CUDART_INF_F;
        }
    };
    const float target = a.us[b] * (residual ? res_total : s_sum[s_end]);
    // every thread walks the range sums: the first range whose inclusive prefix exceeds the
    // target, or the last one with any mass if rounding leaves none
    int rsel = -1, last_r = 0;
    float before_range = 0.f, before_last = 0.f;
    {
        const int nr = residual ? kWarps : a.slices * kWarps;
        if (tid < nr) {          // one range sum per thread, brought to the row's maximum
            if (residual) {
                s_rsum[tid] = s_scan[tid];
            } else {
                const float2 t = __ldcg(a.part + ((size_t)b * N + s_end) * a.slices * kWarps + tid);
                s_rsum[tid] = t.x == -CUDART_INF_F ? 0.f : t.y * ex2((t.x - mx) * kLog2e);
            }
        }
        __syncthreads();
        float run = 0.f;
        for (int r = 0; r < nr; ++r) {
            const float sr = s_rsum[r];
            if (rsel < 0 && run + sr > target) { rsel = r; before_range = run; }
            if (sr > 0.f) { last_r = r; before_last = run; }
            run += sr;
        }
    }
    __syncthreads();   // s_scan is reused below
    const bool crossing = rsel >= 0;
    if (!crossing) { rsel = last_r; before_range = before_last; }
    if (tid == 0) s_pick = kNone;
    int r0, r1;
    if (residual) {
        r0 = min(rsel * rper, rn) * runit;
        r1 = min(rsel * rper + rper, rn) * runit;
    } else {
        range_of(V, a.slices, a.vec, rsel, r0, r1);
    }
    const int per = (r1 - r0 + kThreads - 1) / kThreads;
    const int j0 = min(r0 + tid * per, r1), j1 = min(j0 + per, r1);
    float piece = 0.f;
    int last_pos = -1;
    for (int c0 = j0; c0 < j1; c0 += 16) {
        float xv[16], yv[16];
        load16(x, a.vec != 0, c0, j1, xv);
        if (residual) load16(y, a.dvec != 0, c0, j1, yv);
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const float e = weight(xv[k], residual ? yv[k] : 0.f);
            piece += e;
            if (e > 0.f) last_pos = c0 + k;
        }
    }
    float inc = piece;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) s_scan[warp] = inc;
    __syncthreads();
    float base = before_range;
#pragma unroll
    for (int w = 0; w < kWarps; ++w)
        if (w < warp) base += s_scan[w];
    inc += base;
    // The pieces partition the cumulative axis exactly: a piece begins where the one before it
    // ends (its predecessor's inclusive value, not inc - piece, which rounding could move past a
    // target that the predecessor had not reached).  The first piece whose inclusive value exceeds
    // the target holds the crossing.
    float before = __shfl_up_sync(0xFFFFFFFFu, inc, 1);
    if (lane == 0) before = base;
    if (crossing && inc > target) atomicMin(&s_pick, tid);
    __syncthreads();
    const int first = s_pick;           // kNone: rounding left no crossing in this range
    __syncthreads();
    if (tid == first) {
        float cum = before;
        int pick = -1;
        for (int c0 = j0; c0 < j1 && pick < 0; c0 += 16) {
            float xv[16], yv[16];
            load16(x, a.vec != 0, c0, j1, xv);
            if (residual) load16(y, a.dvec != 0, c0, j1, yv);
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                cum += weight(xv[k], residual ? yv[k] : 0.f);
                if (pick < 0 && cum > target) pick = c0 + k;
            }
        }
        s_pick = pick;                  // -1: the serial sum stayed at or below the target
    }
    // without a crossing the draw is the last entry with any mass at or before that piece (in
    // the whole range if no piece claimed the target)
    int lp = (first == kNone || tid <= first) ? last_pos : -1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lp = max(lp, __shfl_xor_sync(0xFFFFFFFFu, lp, o));
    if (lane == 0) s_red[warp] = lp;
    __syncthreads();
    if (tid == 0) {
        int pick = first == kNone ? -1 : s_pick;
        if (pick < 0)
            for (int w = 0; w < kWarps; ++w) pick = max(pick, s_red[w]);
        if (s_m < a.Tcap && GSD_IN_BOUNDS(s_m >= 0 && pick < V, a.status)) out_tok[s_m] = pick;
    }
}

// First launch: one CTA per (slice, row) streams its part of the row and leaves the warps'
// (maximum, sum) pairs in scratch.
template <bool kVec>
__global__ void __launch_bounds__(kThreads) accept_sampled_kernel(SampledArgs a) {
    // the per-sequence pass (a programmatic dependent launch) may become resident as CTAs retire
    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int row = blockIdx.y;  // b * N + n
    const int slice = blockIdx.x;
    const float* x = a.logits + (size_t)row * a.V;
    Ms r{-CUDART_INF_F, 0.f};
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int lo, hi;
    range_of(a.V, a.slices, kVec ? 1 : 0, slice * kWarps + warp, lo, hi);
    if (kVec) {
        const float4* x4 = reinterpret_cast<const float4*>(x);
        const int a1 = hi >> 2;
        int i = (lo >> 2) + lane;
        // four independent 16-byte loads in flight per thread, each a 512-byte run per warp
        for (; i + 3 * 32 < a1; i += 4 * 32) {
            const float4 r0 = __ldcs(x4 + i), r1 = __ldcs(x4 + i + 32);
            const float4 r2 = __ldcs(x4 + i + 64), r3 = __ldcs(x4 + i + 96);
            take16(r, r0, r1, r2, r3);
        }
        for (; i < a1; i += 32) {
            const float4 t = __ldcs(x4 + i);
            take1(r, t.x); take1(r, t.y); take1(r, t.z); take1(r, t.w);
        }
    } else {
        for (int i = lo + lane; i < hi; i += 32) take1(r, __ldcs(x + i));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Ms t;
        t.m = __shfl_xor_sync(0xFFFFFFFFu, r.m, o);
        t.s = __shfl_xor_sync(0xFFFFFFFFu, r.s, o);
        r = combine(r, t);
    }
    if (lane == 0) a.part[((size_t)row * a.slices + slice) * kWarps + warp] = make_float2(r.m, r.s);
}

// Second launch: one CTA per sequence does the rest (statistics per node, step tests, longest
// path, regenerated token) once every pair of the first launch is visible.
__global__ void __launch_bounds__(kThreads, 1) accept_sampled_tail_kernel(SampledArgs a) {
    finish_sequence(a, blockIdx.x);      // (waits for the first launch inside, as late as it can)
}

int pick_slices(long rows, int V, int sm_count) {
    // enough CTAs to cover the machine a few times over, slices of at least 4096 floats
    int slices = 1;
    const long want = (long)sm_count * 8;
    while (rows * slices < want && (V / (slices * 2)) >= 4096 && slices * 2 <= kMaxSlices) slices *= 2;
    return slices;
}

}  // namespace
}  // namespace gsd

extern "C" size_t gsd_accept_sampled_workspace_bytes(const gsd_accept_params* p) {
    if (!p || p->B < 1 || p->N < 1 || p->N > GSD_MAX_NODES) return 0;
    return gsd::align_up((size_t)p->B * p->N * gsd::kMaxSlices * gsd::kWarps * 8, 256);
}

extern "C" int gsd_accept_sampled(const float* logits, const int32_t* draft_tokens,
                                  const int32_t* parent_ptr, const int32_t* parent_idx,
                                  const float* draft_logits, const float* draft_q,
                                  const float* u_accept, const float* u_sample,
                                  int32_t* accepted_tokens, int32_t* accepted_len,
                                  int32_t* accepted_nodes, const gsd_accept_params* p,
                                  void* workspace, size_t workspace_bytes, int32_t* status,
                                  void* stream) {
    using namespace gsd;
    if (!p || !logits || !draft_tokens || !parent_ptr || !parent_idx || !draft_q || !u_accept ||
        !u_sample || !accepted_tokens || !accepted_len)
        return GSD_ERR_NULL_POINTER;
    if (p->B < 1 || p->N < 1 || p->N > GSD_MAX_NODES || p->V < 1 || p->Ecap < 1 || p->Tcap < 1)
        return GSD_ERR_BAD_SHAPE;
    if ((long long)p->B * p->N > (1ll << 30)) return GSD_ERR_BAD_SHAPE;
    if (((uintptr_t)logits & 3u) != 0 || ((uintptr_t)draft_logits & 3u) != 0) return GSD_ERR_MISALIGNED;
    const size_t need = gsd_accept_sampled_workspace_bytes(p);
    if (!workspace || workspace_bytes < need) return GSD_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 7u) != 0) return GSD_ERR_MISALIGNED;
    DeviceInfo di;
    if (device_info(&di) != 0) return GSD_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;

    SampledArgs a;
    a.logits = logits; a.dlogits = draft_logits; a.tok = draft_tokens; a.pptr = parent_ptr; a.pidx = parent_idx;
    a.q = draft_q; a.u = u_accept; a.us = u_sample;
    a.out_tok = accepted_tokens; a.out_len = accepted_len; a.out_nodes = accepted_nodes;
    a.part = (float2*)workspace;
    a.status = status;
    a.B = p->B; a.N = p->N; a.V = p->V; a.Ecap = p->Ecap; a.Tcap = p->Tcap;
    const bool vec = (p->V % 4 == 0) && (((uintptr_t)logits & 15u) == 0);
    a.slices = pick_slices((long)p->B * p->N, p->V, di.sm_count);
    a.vec = vec ? 1 : 0;
    a.dvec = (draft_logits && (p->V % 4 == 0) && (((uintptr_t)draft_logits & 15u) == 0)) ? 1 : 0;

    // every pair is written before it is read: nothing in the scratch has to start at zero.
    // grid.y holds at most 65535 rows: larger problems go out in blocks of whole sequences.
    const int seq_per = 65535 / p->N;
    for (int b0 = 0; b0 < p->B; b0 += seq_per) {
        const int nb = (p->B - b0 < seq_per) ? p->B - b0 : seq_per;
        SampledArgs s = a;
        s.logits += (size_t)b0 * p->N * p->V; s.tok += (size_t)b0 * p->N;
        if (s.dlogits) s.dlogits += (size_t)b0 * p->N * p->V;
        s.pptr += (size_t)b0 * (p->N + 1); s.pidx += (size_t)b0 * p->Ecap;
        s.q += (size_t)b0 * p->N; s.u += (size_t)b0 * p->N; s.us += b0;
        s.out_tok += (size_t)b0 * p->Tcap; s.out_len += b0;
        if (s.out_nodes) s.out_nodes += (size_t)b0 * p->Tcap;
        s.part += (size_t)b0 * p->N * a.slices * kWarps; s.B = nb;
        const dim3 grid(a.slices, (unsigned)(nb * p->N));
        if (vec) accept_sampled_kernel<true><<<grid, kThreads, 0, st>>>(s);
        else accept_sampled_kernel<false><<<grid, kThreads, 0, st>>>(s);
        GSD_CUDA_TRY(cudaGetLastError());
        cudaLaunchAttribute attr[1];
        dependent_launch_attr(attr);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)nb);
        cfg.blockDim = dim3(kThreads);
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        GSD_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_sampled_tail_kernel, s));
    }
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}
