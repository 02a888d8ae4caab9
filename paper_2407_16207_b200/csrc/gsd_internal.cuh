// Internal declarations shared by the translation units of libgsd (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "gsd.h"

namespace gsd {

void set_cuda_error(cudaError_t e, const char* where);
void set_error_text(const char* text);

#define GSD_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) {                            \
            ::gsd::set_cuda_error(e__, #expr);               \
            return GSD_ERR_CUDA;                             \
        }                                                    \
    } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct DeviceInfo {
    int sm_count;
    int max_smem_optin;
};
// Properties of the current device (cached per device ordinal).
int device_info(DeviceInfo* out);

// ---- verify-attention back ends (they validate nothing: the API layer did) ----
struct AttnArgs {
    const void *q, *k_cache, *v_cache, *draft_k, *draft_v;
    const uint32_t* mask;
    const int32_t* seq_lens;
    void* out;
    int B, N, Hq, Hkv, D, Lmax, G, W;
    float scale_log2;   // softmax_scale * log2(e)
    int num_splits;
    void* workspace;
    int32_t* status;
    cudaStream_t stream;
};

// split planning shared by the back ends and the workspace query
int attn_pick_kernel(const gsd_attn_params* p);                 // GSD_ATTN_MMA or GSD_ATTN_TCGEN05
int attn_auto_splits(const gsd_attn_params* p, int kernel, int sm_count);
size_t attn_partial_bytes(const gsd_attn_params* p, int splits);

int launch_attn_mma(const AttnArgs& a);
int launch_attn_tcgen05(const AttnArgs& a);
bool attn_tcgen05_supports(int D, int G);
int launch_attn_merge(const AttnArgs& a);

}  // namespace gsd
