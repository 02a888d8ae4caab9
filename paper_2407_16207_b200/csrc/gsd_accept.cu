// gsd_accept: greedy verification (vocabulary argmax per draft node) and the longest
// accepted root path through the draft DAG (Sec. 3 deterministic verification and the
// rejection cascade; Sec. 4.1 longest-path selection).
//
// One launch.  Grid (splits, B*N): each CTA streams one slice of one logits row with
// 16-byte loads and reduces (value, index) pairs; slices of a row meet in a packed 64-bit
// atomicMax.  The CTA that finishes last for a sequence runs the path pass for it
// (gsd_path.cuh: level-synchronous relaxation of best[v] = 1 + max over accepted parents,
// selection of the end node, backtracking, emission).
#include "gsd_internal.cuh"
#include "gsd_path.cuh"
#include <math_constants.h>

namespace gsd {
namespace {

constexpr int kThreads = kPathThreads;
constexpr int kNone = 0x7FFFFFFF;

struct Best {
    float v;
    int i;
};

__device__ __forceinline__ void take(Best& b, float v, int i) {
    if (v > b.v) {  // false for NaN; strict: an equal later value never replaces
        b.v = v;
        b.i = i;
    }
}

__device__ __forceinline__ Best better(Best a, Best b) {
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

// monotone map of non-NaN floats to unsigned (with -0 folded onto +0)
__device__ __forceinline__ unsigned ordered_bits(float v) {
    if (v == 0.0f) v = 0.0f;
    unsigned u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ unsigned long long pack_key(float v, int i) {
    return ((unsigned long long)ordered_bits(v) << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)i);
}

__device__ __forceinline__ int key_index(unsigned long long key) {
    return key == 0ull ? 0 : (int)(0xFFFFFFFFu - (unsigned)(key & 0xFFFFFFFFull));
}

__device__ Best block_best(Best b, Best* sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Best t;
        t.v = __shfl_xor_sync(0xFFFFFFFFu, b.v, o);
        t.i = __shfl_xor_sync(0xFFFFFFFFu, b.i, o);
        b = better(b, t);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) sh[warp] = b;
    __syncthreads();
    if (warp == 0) {
        b = lane < (kThreads / 32) ? sh[lane] : Best{-CUDART_INF_F, kNone};
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) {
            Best t;
            t.v = __shfl_xor_sync(0xFFFFFFFFu, b.v, o);
            t.i = __shfl_xor_sync(0xFFFFFFFFu, b.i, o);
            b = better(b, t);
        }
        if (lane == 0) sh[0] = b;
    }
    __syncthreads();
    b = sh[0];
    __syncthreads();
    return b;
}

struct AcceptArgs {
    const float* logits;
    const int32_t* tok;
    const int32_t* pptr;
    const int32_t* pidx;
    int32_t* out_tok;
    int32_t* out_len;
    int32_t* out_nodes;
    unsigned long long* keys;  // [B*N], zeroed before the launch
    unsigned* done;            // [B], zeroed before the launch
    int32_t* status;
    int B, N, V, Ecap, Tcap, splits;
};

__device__ void path_pass(const AcceptArgs& a, int b) {
    __shared__ int s_amax[GSD_MAX_NODES];
    const int N = a.N, tid = threadIdx.x;
    // the keys were written by other CTAs: read them past L1.  (No barrier of its own: the path
    // routine fetches the graph first and meets at a barrier before any step is tested, so the
    // two trips to memory overlap.)
    for (int v = tid; v < N; v += kThreads) s_amax[v] = key_index(__ldcg(a.keys + (size_t)b * N + v));
    const int32_t* tok = a.tok + (size_t)b * N;
    PathIo io;
    io.tok = tok;
    io.pptr = a.pptr + (size_t)b * (N + 1);
    io.pidx = a.pidx + (size_t)b * a.Ecap;
    io.out_tok = a.out_tok + (size_t)b * a.Tcap;
    io.out_nodes = a.out_nodes ? a.out_nodes + (size_t)b * a.Tcap : nullptr;
    io.out_len = a.out_len + b;
    io.status = a.status;
    io.N = N; io.V = a.V; io.Ecap = a.Ecap; io.Tcap = a.Tcap;
    // a step parent -> v is accepted iff v's token is what the target model would emit after the parent
    const PathResult res = longest_accepted_path<false>(io, 0u, [&](int p, int v) { return tok[v] == s_amax[p]; });
    // the target model's own next token
    if (tid == 0 && res.edges < a.Tcap && GSD_IN_BOUNDS(res.end >= 0 && res.end < N && res.edges >= 0, a.status))
        io.out_tok[res.edges] = s_amax[res.end];
}

// Zeroes scratch words.  The kernel that uses them is launched as a programmatic dependent: it
// may start streaming its input at once and only waits for these zeros before its first atomic.
__global__ void clear_words_kernel(unsigned* words, int n) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) words[i] = 0u;
}

template <bool kVec>
__global__ void __launch_bounds__(kThreads) accept_kernel(AcceptArgs a) {
    __shared__ Best sh[kThreads / 32];
    __shared__ int s_last;
    const int row = blockIdx.y;  // b * N + n
    const int split = blockIdx.x;
    const float* x = a.logits + (size_t)row * a.V;
    Best best{-CUDART_INF_F, kNone};
    int lo, hi;  // element range of this slice
    if (kVec) {
        const int nvec = a.V >> 2;
        const int per = (nvec + a.splits - 1) / a.splits;
        const int v0 = min(split * per, nvec), v1 = min(v0 + per, nvec);
        lo = v0 * 4;
        hi = v1 * 4;
        const float4* x4 = reinterpret_cast<const float4*>(x);
        int i = v0 + threadIdx.x;
        // four independent 16-byte loads in flight per thread
        for (; i + 3 * kThreads < v1; i += 4 * kThreads) {
            float4 r0 = __ldcs(x4 + i), r1 = __ldcs(x4 + i + kThreads);
            float4 r2 = __ldcs(x4 + i + 2 * kThreads), r3 = __ldcs(x4 + i + 3 * kThreads);
            int e = i * 4;
            take(best, r0.x, e); take(best, r0.y, e + 1); take(best, r0.z, e + 2); take(best, r0.w, e + 3);
            e += 4 * kThreads;
            take(best, r1.x, e); take(best, r1.y, e + 1); take(best, r1.z, e + 2); take(best, r1.w, e + 3);
            e += 4 * kThreads;
            take(best, r2.x, e); take(best, r2.y, e + 1); take(best, r2.z, e + 2); take(best, r2.w, e + 3);
            e += 4 * kThreads;
            take(best, r3.x, e); take(best, r3.y, e + 1); take(best, r3.z, e + 2); take(best, r3.w, e + 3);
        }
        for (; i < v1; i += kThreads) {
            float4 r = __ldcs(x4 + i);
            const int e = i * 4;
            take(best, r.x, e); take(best, r.y, e + 1); take(best, r.z, e + 2); take(best, r.w, e + 3);
        }
    } else {
        const int per = (a.V + a.splits - 1) / a.splits;
        lo = min(split * per, a.V);
        hi = min(lo + per, a.V);
        for (int i = lo + threadIdx.x; i < hi; i += kThreads) take(best, __ldcs(x + i), i);
    }
    best = block_best(best, sh);
    if (best.i == kNone) {
        // nothing above -inf in this slice: the lowest non-NaN entry (a -inf), if any, stands
        int first = kNone;
        for (int i = lo + threadIdx.x; i < hi; i += kThreads)
            if (x[i] == x[i]) { first = i; break; }
        Best f{first == kNone ? -CUDART_INF_F : 0.0f, first};  // the value only orders this reduction
        f = block_best(f, sh);
        best.i = f.i;
        best.v = -CUDART_INF_F;
    }
    if (threadIdx.x == 0) {
        // the scratch is zeroed by the launch before this one; everything above ran beside it
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (best.i != kNone && GSD_IN_BOUNDS(row < a.B * a.N && best.i >= 0 && best.i < a.V, a.status))
            atomicMax(a.keys + row, pack_key(best.v, best.i));
        __threadfence();
        const int b = row / a.N;
        const unsigned prev = atomicAdd(a.done + b, 1u);
        s_last = (prev == (unsigned)(a.N * a.splits) - 1u);
    }
    __syncthreads();
    if (s_last) {
        __threadfence();
        path_pass(a, row / a.N);
    }
}

}  // namespace

int launch_clear_words(unsigned* words, int n, cudaStream_t stream) {
    const int blocks = (n + 1023) / 1024;
    clear_words_kernel<<<blocks < 64 ? blocks : 64, 256, 0, stream>>>(words, n);
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}

}  // namespace gsd

extern "C" size_t gsd_accept_workspace_bytes(const gsd_accept_params* p) {
    if (!p || p->B < 1 || p->N < 1 || p->N > GSD_MAX_NODES) return 0;
    return gsd::align_up((size_t)p->B * p->N * 8 + (size_t)p->B * 4, 256);
}

extern "C" int gsd_accept(const float* logits, const int32_t* draft_tokens,
                          const int32_t* parent_ptr, const int32_t* parent_idx,
                          int32_t* accepted_tokens, int32_t* accepted_len, int32_t* accepted_nodes,
                          const gsd_accept_params* p, void* workspace, size_t workspace_bytes,
                          int32_t* status, void* stream) {
    using namespace gsd;
    if (!p || !logits || !draft_tokens || !parent_ptr || !parent_idx || !accepted_tokens ||
        !accepted_len)
        return GSD_ERR_NULL_POINTER;
    if (p->B < 1 || p->N < 1 || p->N > GSD_MAX_NODES || p->V < 1 || p->Ecap < 1 || p->Tcap < 1)
        return GSD_ERR_BAD_SHAPE;
    if ((long long)p->B * p->N > (1ll << 30)) return GSD_ERR_BAD_SHAPE;
    if (((uintptr_t)logits & 3u) != 0) return GSD_ERR_MISALIGNED;
    const size_t need = gsd_accept_workspace_bytes(p);
    if (!workspace || workspace_bytes < need) return GSD_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 7u) != 0) return GSD_ERR_MISALIGNED;
    DeviceInfo di;
    if (device_info(&di) != 0) return GSD_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;

    AcceptArgs a;
    a.logits = logits; a.tok = draft_tokens; a.pptr = parent_ptr; a.pidx = parent_idx;
    a.out_tok = accepted_tokens; a.out_len = accepted_len; a.out_nodes = accepted_nodes;
    a.keys = (unsigned long long*)workspace;
    a.done = (unsigned*)((char*)workspace + (size_t)p->B * p->N * 8);
    a.status = status;
    a.B = p->B; a.N = p->N; a.V = p->V; a.Ecap = p->Ecap; a.Tcap = p->Tcap;
    const bool vec = (p->V % 4 == 0) && (((uintptr_t)logits & 15u) == 0);
    // enough CTAs to cover the machine a few times over, slices of at least 4096 floats
    const long rows = (long)p->B * p->N;
    int splits = 1;
    const long want = (long)di.sm_count * 8;
    while (rows * splits < want && (p->V / (splits * 2)) >= 4096) splits *= 2;
    a.splits = splits;

    if (launch_clear_words((unsigned*)workspace, p->B * p->N * 2 + p->B, st) != GSD_OK) return GSD_ERR_CUDA;
    cudaLaunchAttribute attr[1];
    dependent_launch_attr(attr);
    // grid.y holds at most 65535 rows: larger problems go out in blocks of whole sequences
    // so that the per-sequence completion counter still works
    const int seq_per = 65535 / p->N;
    for (int b0 = 0; b0 < p->B; b0 += seq_per) {
        const int nb = (p->B - b0 < seq_per) ? p->B - b0 : seq_per;
        AcceptArgs s = a;
        s.logits += (size_t)b0 * p->N * p->V; s.tok += (size_t)b0 * p->N;
        s.pptr += (size_t)b0 * (p->N + 1); s.pidx += (size_t)b0 * p->Ecap;
        s.out_tok += (size_t)b0 * p->Tcap; s.out_len += b0;
        if (s.out_nodes) s.out_nodes += (size_t)b0 * p->Tcap;
        s.keys += (size_t)b0 * p->N; s.done += b0; s.B = nb;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(splits, (unsigned)(nb * p->N));
        cfg.blockDim = dim3(kThreads);
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (vec) GSD_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_kernel<true>, s));
        else GSD_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_kernel<false>, s));
    }
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}

// ---------------------------------------------------------------------------------------
// gsd_accept_static: the same computation as gsd_accept with the scratch in a fixed array
// that lives in the library image, for callers that cannot hand over device memory.
namespace gsd {
namespace {
// 8 bytes per draft node plus 4 bytes per sequence, for at most GSD_STATIC_MAX_ROWS rows.
// Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_accept_scratch[GSD_STATIC_SCRATCH_BYTES];
}  // namespace
}  // namespace gsd

extern "C" int gsd_accept_static(const float* logits, const int32_t* draft_tokens,
                                 const int32_t* parent_ptr, const int32_t* parent_idx,
                                 int32_t* accepted_tokens, int32_t* accepted_len,
                                 int32_t* accepted_nodes, const gsd_accept_params* p,
                                 int32_t* status, void* stream) {
    using namespace gsd;
    if (!p) return GSD_ERR_NULL_POINTER;
    if (p->B < 1 || p->N < 1 || p->N > GSD_MAX_NODES) return GSD_ERR_BAD_SHAPE;
    if ((long long)p->B * p->N > GSD_STATIC_MAX_ROWS) {
        set_error_text("gsd_accept_static: B*N exceeds GSD_STATIC_MAX_ROWS");
        return GSD_ERR_WORKSPACE;
    }
    const size_t need = gsd_accept_workspace_bytes(p);
    if (need == 0 || need > (size_t)GSD_STATIC_SCRATCH_BYTES) {
        set_error_text("gsd_accept_static: scratch need exceeds GSD_STATIC_SCRATCH_BYTES");
        return GSD_ERR_WORKSPACE;
    }
    // In host code the array's name is only a handle; the device address has to be asked for,
    // once per device, with that device current.
    static void* addr[64] = {};
    int dev = 0;
    GSD_CUDA_TRY(cudaGetDevice(&dev));
    void* ptr = (dev >= 0 && dev < 64) ? addr[dev] : nullptr;
    if (!ptr) {
        GSD_CUDA_TRY(cudaGetSymbolAddress((void**)&ptr, g_accept_scratch));
        if (!ptr) return GSD_ERR_CUDA;
        if (dev >= 0 && dev < 64) addr[dev] = ptr;
    }
    // gsd_accept clears the part of the scratch it uses before every launch
    return gsd_accept(logits, draft_tokens, parent_ptr, parent_idx, accepted_tokens, accepted_len,
                      accepted_nodes, p, ptr, (size_t)GSD_STATIC_SCRATCH_BYTES, status, stream);
}
