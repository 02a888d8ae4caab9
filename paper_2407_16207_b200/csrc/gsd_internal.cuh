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

// Index checks of the checking build (compiled with -DGSD_BOUNDS_CHECK into libgsd_check.so; the
// stand-in for a memory sanitizer): at the places where a kernel forms an index into global
// memory from data or from its work plan, GSD_IN_BOUNDS(condition, status) is the condition
// itself and, when it fails, ORs GSD_DEV_BOUNDS into the status word - the caller skips the
// access, nothing traps.  In the ordinary build it is the constant true and costs nothing.
#ifdef GSD_BOUNDS_CHECK
__device__ __forceinline__ bool note_out_of_bounds(int32_t* status) {
    if (status) atomicOr((unsigned*)status, GSD_DEV_BOUNDS);
    return false;
}
#define GSD_IN_BOUNDS(cond, status) ((cond) ? true : ::gsd::note_out_of_bounds(status))
#else
#define GSD_IN_BOUNDS(cond, status) (true)
#endif

struct DeviceInfo {
    int sm_count;
    int max_smem_optin;
};
// Properties of the current device (cached per device ordinal).
int device_info(DeviceInfo* out);

// ---- work plan of one gsd_verify_attn call ----
// A work item is one row tile (rows_per_item stacked rows) of one (sequence, kv head); item
// index = unit * tiles_per_unit + row tile.  The first items_a items are cut into splits_a
// key ranges, the remaining ones into splits_b; CTAs are numbered group a first.  Only items
// with more than one split own partial-result slots (one per split, numbered in CTA order).
//
// Balanced plan (tcgen05 back end only): the host cannot see the sequence lengths, so for
// batches whose lengths differ a plan made from Lmax leaves CTAs idle.  Here the key tiles of
// all (sequence, kv head) pairs are laid end to end - pair after pair, ceil(len/128) prefix
// tiles plus the draft tiles each - and group g of `ctas / tiles_per_unit` groups takes the
// g-th equal share of that line; CTA r of a group works on row-tile item r of every pair in
// the share.  A small kernel builds the table from seq_lens on the device before the
// attention kernel reads it: per group its units (pair, tile range, partial-result slot or -1
// for a whole pair), and per pair that was cut the run of slots to merge.  Slots are numbered
// along the line, so the pieces of one pair have consecutive slots; a group has at most two
// partial units (its first and last).  CTA r adds r * 2 * groups to a slot of its group.
//
// Per-sequence plan (tcgen05 back end only): a lighter form of the same idea that keeps the
// CTAs of one sequence in step.  Every item of sequence b is cut into nsplit[b] equal key
// ranges, nsplit[b] = its tile count over a common target length (rounded), chosen on the
// device so that the batch makes about `units_wanted` units; units are numbered sequence by
// sequence, range by range, item by item, and CTA k walks units k, k + grid, ...  The heads of
// a sequence then read the same cache rows at the same time, which the head-interleaved cache
// layout rewards (a row of the cache holds all kv heads of a position).
struct PlanDev {
    int items_a, splits_a, splits_b, tiles_per_unit;
    int balanced;       // 1: units come from the table built on the device; 2: per-sequence split counts from the device
};
struct AttnPlan {
    int kernel;         // GSD_ATTN_MMA or GSD_ATTN_TCGEN05
    int rows_per_item;  // 64 (mma.sync back end) or 256 (tcgen05 back end)
    int items;
    int ctas;
    int slots;          // partial-result slots; 0 when nothing is split
    PlanDev dev;
    size_t ws_bytes;
};
// The table of a balanced plan, in the workspace behind the partial results.
struct BalTable {
    int* hdr;       // [0] pairs to merge, [1] tiles on the line, [2] tiles per group
    int2* cta;      // [groups]  (index of the group's first unit, number of units)
    int4* merge;    // [groups]  (pair, first slot, number of slots, -)
    int4* units;    // [pairs + groups]  (pair, first tile, end tile, slot or -1); tiles count the
                    //                   prefix tiles, then ALL draft tiles of the pair
    int* off;       // [B + 1] start of each sequence on the line
};
__host__ __device__ inline void plan_decode(const PlanDev& pl, int cta, int& item, int& split, int& nsplit, int& slot) {
    const int ctas_a = pl.items_a * pl.splits_a;
    if (cta < ctas_a) {
        item = cta / pl.splits_a;
        split = cta - item * pl.splits_a;
        nsplit = pl.splits_a;
        slot = cta;
    } else {
        const int rem = cta - ctas_a;
        const int k = rem / pl.splits_b;
        item = pl.items_a + k;
        split = rem - k * pl.splits_b;
        nsplit = pl.splits_b;
        slot = (pl.splits_a > 1 ? ctas_a : 0) + rem;
    }
}
AttnPlan attn_make_plan(const gsd_attn_params* p, int sm_count);

// ---- verify-attention back ends (they validate nothing: the API layer did) ----
struct AttnArgs {
    const void *q, *k_cache, *v_cache, *draft_k, *draft_v;
    const uint32_t* mask;
    const int32_t* seq_lens;
    void* out;
    int B, N, Hq, Hkv, D, Lmax, G, W;
    float scale_log2;   // softmax_scale * log2(e)
    AttnPlan plan;
    void* workspace;
    int32_t* status;
    cudaStream_t stream;
};

int attn_pick_kernel(const gsd_attn_params* p);                 // GSD_ATTN_MMA or GSD_ATTN_TCGEN05
// partial results: fp32 accumulators [slot][rows_per_item][D], then (max, sum) [slot][rows_per_item][2]
inline size_t plan_part_o_bytes(const AttnPlan& pl, int D) { return align_up((size_t)pl.slots * pl.rows_per_item * D * sizeof(float), 256); }
inline size_t plan_part_ml_bytes(const AttnPlan& pl) { return align_up((size_t)pl.slots * pl.rows_per_item * 2 * sizeof(float), 256); }

// The table of a per-sequence plan, in the workspace behind the partial results.
struct SeqTable {
    int* hdr;        // [0] units of work, [1] tiles of all items, [2] target tiles per unit
    int* nsplit;     // [B]     key ranges per item of the sequence
    int* unit_off;   // [B + 1] first unit of the sequence
    int* slot_off;   // [B + 1] first partial-result slot of the sequence (sequences cut in two or more only)
};
inline size_t plan_bal_bytes(const AttnPlan& pl, int B) {
    if (!pl.dev.balanced) return 0;
    if (pl.dev.balanced == 2) return 256 + 3 * align_up((size_t)(B + 1) * sizeof(int), 256);
    return 256 + align_up((size_t)pl.ctas * sizeof(int2), 256) + align_up((size_t)pl.ctas * sizeof(int4), 256) +
           align_up((size_t)(pl.items + pl.ctas) * sizeof(int4), 256) + align_up((size_t)(B + 1) * sizeof(int), 256);
}
inline BalTable plan_bal_table(const AttnPlan& pl, int D, void* workspace) {
    char* at = (char*)workspace + plan_part_o_bytes(pl, D) + plan_part_ml_bytes(pl);
    BalTable t;
    t.hdr = (int*)at; at += 256;
    t.cta = (int2*)at; at += align_up((size_t)pl.ctas * sizeof(int2), 256);
    t.merge = (int4*)at; at += align_up((size_t)pl.ctas * sizeof(int4), 256);
    t.units = (int4*)at; at += align_up((size_t)(pl.items + pl.ctas) * sizeof(int4), 256);
    t.off = (int*)at;
    return t;
}

inline SeqTable plan_seq_table(const AttnPlan& pl, int D, int B, void* workspace) {
    char* at = (char*)workspace + plan_part_o_bytes(pl, D) + plan_part_ml_bytes(pl);
    const size_t row = align_up((size_t)(B + 1) * sizeof(int), 256);
    SeqTable t;
    t.hdr = (int*)at; at += 256;
    t.nsplit = (int*)at; at += row;
    t.unit_off = (int*)at; at += row;
    t.slot_off = (int*)at;
    return t;
}
constexpr int kSeqPlanWaves = 2;              // units a per-sequence plan aims at, per resident CTA
constexpr int kSeqPlanMaxSplit = 32;

int launch_attn_plan(const AttnArgs& a);      // plans made on the device only: builds the table
int launch_attn_mma(const AttnArgs& a);
int launch_attn_tcgen05(const AttnArgs& a);
bool attn_tcgen05_supports(int D, int G);
int launch_attn_merge(const AttnArgs& a);
// test hook behind gsd_debug_attn_wait (process-wide; 0 restores the default limit)
void debug_attn_wait(unsigned long long limit_ns, int withhold_first_k);

// ---- scratch words that must start at zero ----
// Enqueues a small kernel that zeroes `n` 32-bit words and lets the next launch on the stream
// start beside it.  That next kernel has to be launched with the attribute set up by
// dependent_launch_attr() and to execute griddepcontrol.wait before it first touches the words.
int launch_clear_words(unsigned* words, int n, cudaStream_t stream);
inline void dependent_launch_attr(cudaLaunchAttribute* attr) {
    attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr->val.programmaticStreamSerializationAllowed = 1;
}

}  // namespace gsd
