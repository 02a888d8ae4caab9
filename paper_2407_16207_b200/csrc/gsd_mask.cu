// gsd_build_mask: ancestor bitmask of a draft DAG from its parent lists in CSR form, i.e. what
// "a token may only attend to its ancestor nodes" (tree attention, Sec. 4.1) means for the
// merged token graph (Sec. 5.3): bit j of row n is set iff j == n or n can be reached from j.
//
// One CTA per sequence keeps the N x W word matrix in shared memory and relaxes
// row[v] |= OR over parents p of row[p] level-synchronously until nothing changes (at most
// longest-path + 1 rounds; parents precede children, so one round settles one more level).
// Words only ever gain bits, so the in-place update needs no second buffer.
#include "gsd_internal.cuh"

namespace gsd {
namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
build_mask_kernel(const int32_t* __restrict__ parent_ptr, const int32_t* __restrict__ parent_idx,
                  uint32_t* __restrict__ mask, int N, int W, int Ecap, int32_t* status) {
    extern __shared__ uint32_t s_rows_raw[];
    volatile uint32_t* rows = s_rows_raw;
    const int b = blockIdx.x, tid = threadIdx.x;
    const int32_t* pp = parent_ptr + (size_t)b * (N + 1);
    const int32_t* pi = parent_idx + (size_t)b * Ecap;
    const int tasks = N * W;
    for (int t = tid; t < tasks; t += kThreads) {
        const int v = t / W, w = t - v * W;
        rows[t] = (w == (v >> 5)) ? (1u << (v & 31)) : 0u;
    }
    __syncthreads();
    unsigned flags = 0;
    for (int round = 0; round < N; ++round) {
        int changed = 0;
        for (int t = tid; t < tasks; t += kThreads) {
            const int v = t / W, w = t - v * W;
            int e0 = pp[v], e1 = pp[v + 1];
            if (e0 < 0 || e1 > Ecap || e0 > e1) {
                flags |= GSD_DEV_BAD_CSR;
                continue;
            }
            uint32_t acc = rows[t];
            const uint32_t before = acc;
            for (int e = e0; e < e1; ++e) {
                const int p = pi[e];
                if (p < 0 || p >= v) {
                    flags |= GSD_DEV_BAD_CSR;
                    continue;
                }
                acc |= rows[p * W + w];
            }
            if (acc != before) {
                rows[t] = acc;
                changed = 1;
            }
        }
        if (!__syncthreads_or(changed)) break;
    }
    uint32_t* out = mask + (size_t)b * tasks;
    for (int t = tid; t < tasks; t += kThreads) out[t] = rows[t];
    if (flags && status) atomicOr((unsigned*)status, flags);
}

}  // namespace
}  // namespace gsd

extern "C" int gsd_build_mask(const int32_t* parent_ptr, const int32_t* parent_idx,
                              uint32_t* ancestor_mask, int32_t B, int32_t N, int32_t Ecap,
                              int32_t* status, void* stream) {
    using namespace gsd;
    if (!parent_ptr || !parent_idx || !ancestor_mask) return GSD_ERR_NULL_POINTER;
    if (B < 1 || B > 65535 * 32 || N < 1 || N > GSD_MAX_NODES || Ecap < 1) return GSD_ERR_BAD_SHAPE;
    const int W = (N + 31) / 32;
    const size_t smem = (size_t)N * W * sizeof(uint32_t);   // at most 32 KB
    build_mask_kernel<<<B, kThreads, smem, (cudaStream_t)stream>>>(parent_ptr, parent_idx, ancestor_mask, N, W,
                                                                  Ecap, status);
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}
