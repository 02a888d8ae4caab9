// gsd_verify_attn, warp-level tensor-core back end (mma.sync m16n8k16 bf16, fp32
// accumulate) and the split-KV merge pass.
//
// Tree attention over the flattened token graph (Sec. 4.1): every draft node attends to
// the committed prefix held in the KV cache (Sec. 4.2) and to the draft nodes named by its
// ancestor bitmask.  For one (sequence, kv head) the G = Hq/Hkv query heads of all N nodes
// are stacked into R = N*G rows (row r = node r / G, head r % G) so that K and V are read
// once per row tile.
//
// Grid: one CTA per (work item, key-range split) of the call's plan.  A CTA of 4 warps owns
// 64 stacked rows and walks its share of the key tiles (64 keys each; prefix tiles first, then draft tiles) with a
// two-stage cp.async pipeline.  Rows of the cache at positions >= seq_lens[b] and draft
// rows >= N are zero-filled by the copy itself, so junk (even NaN patterns) never reaches
// the arithmetic.  Draft tiles whose mask words are all zero for the CTA's rows are
// skipped.  With one split the CTA normalises and stores bf16; otherwise it stores the
// unnormalised fp32 accumulator with (running max, running sum) and the merge pass
// combines the splits.
#include "gsd_internal.cuh"
#include <cuda_bf16.h>
#include <math_constants.h>

namespace gsd {
namespace {

constexpr int BM = 64;   // stacked rows per CTA
constexpr int BN = 64;   // keys per tile
constexpr int kThreads = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

// 16-byte async copy; src_bytes == 0 writes zeros and reads nothing
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte chunk `chunk` of row `row` in a [rows][D] bf16 tile whose chunks
// are XOR-swizzled by the row so that ldmatrix reads hit distinct banks
template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

struct MmaParams {
    const __nv_bfloat16 *q, *k_cache, *v_cache, *draft_k, *draft_v;
    const uint32_t* mask;
    const int32_t* seq_lens;
    __nv_bfloat16* out;
    float* part_o;   // [slot][64][D]
    float* part_ml;  // [slot][64][2]
    PlanDev plan;
    int32_t* status;
    int B, N, Hq, Hkv, Lmax, G, W, R;
    int slots;       // partial-result slots of the plan
    float scale_log2;
};

template <int D>
__global__ void __launch_bounds__(kThreads) attn_mma_kernel(MmaParams p) {
    constexpr int CH = D / 8;              // 16-byte chunks per row
    constexpr int TILE = BN * D * 2;       // bytes of one K or V tile
    constexpr int KS = D / 16;             // k-steps of the QK^T product
    constexpr int NT = BN / 8;             // score n-tiles per warp
    constexpr int DT = D / 8;              // output n-tiles per warp
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sK[2] = {smem, smem + 2 * TILE};
    unsigned char* sV[2] = {smem + TILE, smem + 3 * TILE};
    __shared__ unsigned s_live;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int item, split, nsplit, slot;
    plan_decode(p.plan, blockIdx.x, item, split, nsplit, slot);
    const int unit = item / p.plan.tiles_per_unit;   // b * Hkv + c
    const int row0 = (item % p.plan.tiles_per_unit) * BM;
    const int b = unit / p.Hkv, c = unit % p.Hkv;
    const int N = p.N, G = p.G, R = p.R;

    int L = p.seq_lens[b];
    if (L < 0 || L > p.Lmax) {
        if (tid == 0 && p.status) atomicOr((unsigned*)p.status, GSD_DEV_BAD_SEQ_LEN);
        L = L < 0 ? 0 : p.Lmax;
    }
    const int nPT = (L + BN - 1) / BN, nDT = (N + BN - 1) / BN;
    const int T = nPT + nDT;
    const int per = (T + nsplit - 1) / nsplit;
    const int t_begin = min(split * per, T), t_end = min(t_begin + per, T);

    // which draft tiles hold at least one visible key for this CTA's rows
    if (tid == 0) s_live = 0;
    __syncthreads();
    {
        unsigned live = 0;
        const int r = row0 + tid;
        if (tid < BM && r < R) {
            const uint32_t* mrow = p.mask + ((size_t)b * N + r / G) * p.W;
            for (int w = 0; w < p.W; ++w) {
                uint32_t word = mrow[w];
                if (w == p.W - 1 && (N & 31)) word &= (1u << (N & 31)) - 1u;
                if (word) live |= 1u << (w >> 1);
            }
        }
        live = __reduce_or_sync(0xFFFFFFFFu, live);
        if (lane == 0 && live) atomicOr(&s_live, live);
    }

    // ---- Q tile -> smem (borrowing the second V stage) -> A fragments
    {
        unsigned char* sQ = sV[1];
        for (int i = tid; i < BM * CH; i += kThreads) {
            const int r = i / CH, ch = i % CH;
            const int row = row0 + r;
            const bool ok = row < R;
            const int n = ok ? row / G : 0, g = ok ? row % G : 0;
            const __nv_bfloat16* src = p.q + (((size_t)b * N + n) * p.Hq + c * G + g) * D + ch * 8;
            cp_async16(smem_u32(sQ + tile_off<D>(r, ch)), src, ok ? 16 : 0);
        }
        cp_async_commit();
    }
    cp_async_wait<0>();
    __syncthreads();
    const unsigned live_tiles = s_live;
    uint32_t qf[KS][4];
    {
        unsigned char* sQ = sV[1];
        const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
            ldmatrix_x4(qf[ks], smem_u32(sQ + tile_off<D>(r, ks * 2 + (lane >> 4))));
    }
    __syncthreads();   // Q has been read: the stage may be overwritten

    auto tile_live = [&](int t) -> bool {
        return t < nPT || ((live_tiles >> (t - nPT)) & 1u);
    };
    auto load_tile = [&](int t, int stage) {
        const bool draft = t >= nPT;
        const int key0 = (draft ? t - nPT : t) * BN;
        const int limit = draft ? N : L;
        const __nv_bfloat16* kb = draft ? p.draft_k + ((size_t)b * N * p.Hkv + c) * D
                                        : p.k_cache + ((size_t)b * p.Lmax * p.Hkv + c) * D;
        const __nv_bfloat16* vb = draft ? p.draft_v + ((size_t)b * N * p.Hkv + c) * D
                                        : p.v_cache + ((size_t)b * p.Lmax * p.Hkv + c) * D;
        const size_t rstride = (size_t)p.Hkv * D;
        for (int i = tid; i < BN * CH; i += kThreads) {
            const int r = i / CH, ch = i % CH;
            const int key = key0 + r;
            const bool ok = key < limit;
            const size_t off = (size_t)(ok ? key : 0) * rstride + ch * 8;
            cp_async16(smem_u32(sK[stage] + tile_off<D>(r, ch)), kb + off, ok ? 16 : 0);
            cp_async16(smem_u32(sV[stage] + tile_off<D>(r, ch)), vb + off, ok ? 16 : 0);
        }
    };
    auto next_live = [&](int t) -> int {
        while (t < t_end && !tile_live(t)) ++t;
        return t;
    };

    float o[DT][4];
#pragma unroll
    for (int i = 0; i < DT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F};
    float l_run[2] = {0.f, 0.f};

    // the two rows this thread holds in every accumulator fragment
    const int rloc[2] = {warp * 16 + (lane >> 2), warp * 16 + (lane >> 2) + 8};
    const bool rvalid[2] = {row0 + rloc[0] < R, row0 + rloc[1] < R};

    int t = next_live(t_begin);
    if (t < t_end) load_tile(t, 0);
    cp_async_commit();
    int stage = 0;
    while (t < t_end) {
        const int t_next = next_live(t + 1);
        if (t_next < t_end) load_tile(t_next, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();

        // ---- S = Q K^T for 16 rows x 64 keys
        float s[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int kp = 0; kp < KS / 2; ++kp) {
                uint32_t kf[4];
                ldmatrix_x4(kf, smem_u32(sK[stage] + tile_off<D>(nt * 8 + (lane & 7), kp * 4 + (lane >> 3))));
                mma_bf16(s[nt], qf[kp * 2], kf[0], kf[1]);
                mma_bf16(s[nt], qf[kp * 2 + 1], kf[2], kf[3]);
            }
        }

        // ---- visibility: key index inside the prefix, mask bits inside the draft block
        const bool draft = t >= nPT;
        const int key0 = (draft ? t - nPT : t) * BN;
        if (draft) {
            // lanes 0..31 fetch (row = lane / 2, word = lane % 2) of this warp's 16 rows; the
            // owners of a row then pick their two words up by shuffle
            const int mr = row0 + warp * 16 + (lane >> 1);
            const int wi = (key0 >> 5) + (lane & 1);
            uint32_t word = 0;
            if (mr < R && wi < p.W) word = p.mask[((size_t)b * N + mr / G) * p.W + wi];
            uint32_t mw[2][2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int src_row = (lane >> 2) + h * 8;
                mw[h][0] = __shfl_sync(0xFFFFFFFFu, word, src_row * 2);
                mw[h][1] = __shfl_sync(0xFFFFFFFFu, word, src_row * 2 + 1);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = nt * 8 + (lane & 3) * 2 + (e & 1);
                    const int h = e >> 1;
                    const uint32_t w = (col >> 5) ? mw[h][1] : mw[h][0];
                    const bool vis = ((w >> (col & 31)) & 1u) && (key0 + col < N) && rvalid[h];
                    s[nt][e] = vis ? s[nt][e] * p.scale_log2 : -CUDART_INF_F;
                }
            }
        } else {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = nt * 8 + (lane & 3) * 2 + (e & 1);
                    const bool vis = (key0 + col < L) && rvalid[e >> 1];
                    s[nt][e] = vis ? s[nt][e] * p.scale_log2 : -CUDART_INF_F;
                }
            }
        }

        // ---- online softmax (base 2), fp32
        float alpha[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float mx = -CUDART_INF_F;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) mx = fmaxf(mx, fmaxf(s[nt][h * 2], s[nt][h * 2 + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
            const float m_new = fmaxf(m_run[h], mx);
            const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;  // nothing visible yet
            alpha[h] = exp2f(m_run[h] - m_use);
            m_run[h] = m_new;
            float sum = 0.f;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                s[nt][h * 2] = exp2f(s[nt][h * 2] - m_use);
                s[nt][h * 2 + 1] = exp2f(s[nt][h * 2 + 1] - m_use);
                sum += s[nt][h * 2] + s[nt][h * 2 + 1];
            }
            l_run[h] = l_run[h] * alpha[h] + sum;
        }
#pragma unroll
        for (int dt = 0; dt < DT; ++dt) {
            o[dt][0] *= alpha[0]; o[dt][1] *= alpha[0];
            o[dt][2] *= alpha[1]; o[dt][3] *= alpha[1];
        }

        // ---- O += P V
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
            uint32_t pf[4];
            pf[0] = pack_bf16(s[2 * ks][0], s[2 * ks][1]);
            pf[1] = pack_bf16(s[2 * ks][2], s[2 * ks][3]);
            pf[2] = pack_bf16(s[2 * ks + 1][0], s[2 * ks + 1][1]);
            pf[3] = pack_bf16(s[2 * ks + 1][2], s[2 * ks + 1][3]);
#pragma unroll
            for (int dp = 0; dp < DT / 2; ++dp) {
                uint32_t vf[4];
                const int key = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                ldmatrix_x4_trans(vf, smem_u32(sV[stage] + tile_off<D>(key, dp * 2 + (lane >> 4))));
                mma_bf16(o[dp * 2], pf, vf[0], vf[1]);
                mma_bf16(o[dp * 2 + 1], pf, vf[2], vf[3]);
            }
        }
        __syncthreads();   // every warp is done with this stage before it is refilled
        stage ^= 1;
        t = t_next;
    }
    cp_async_wait<0>();

    // ---- epilogue
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_run[h] += __shfl_xor_sync(0xFFFFFFFFu, l_run[h], 1);
        l_run[h] += __shfl_xor_sync(0xFFFFFFFFu, l_run[h], 2);
    }
    if (nsplit == 1) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (!rvalid[h]) continue;
            const int row = row0 + rloc[h];
            if (!GSD_IN_BOUNDS(b < p.B && c < p.Hkv && row < p.R, p.status)) continue;
            const float inv = l_run[h] > 0.f ? 1.f / l_run[h] : 0.f;
            __nv_bfloat16* dst = p.out + (((size_t)b * N + row / G) * p.Hq + c * G + row % G) * D;
#pragma unroll
            for (int dt = 0; dt < DT; ++dt) {
                const int col = dt * 8 + (lane & 3) * 2;
                *reinterpret_cast<uint32_t*>(dst + col) = pack_bf16(o[dt][h * 2] * inv, o[dt][h * 2 + 1] * inv);
            }
        }
    } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (!rvalid[h]) continue;
            const size_t prow = (size_t)slot * BM + rloc[h];
            if (!GSD_IN_BOUNDS(slot >= 0 && slot < p.slots, p.status)) continue;
            float* dst = p.part_o + prow * D;
#pragma unroll
            for (int dt = 0; dt < DT; ++dt) {
                const int col = dt * 8 + (lane & 3) * 2;
                *reinterpret_cast<float2*>(dst + col) = make_float2(o[dt][h * 2], o[dt][h * 2 + 1]);
            }
            if ((lane & 3) == 0) *reinterpret_cast<float2*>(p.part_ml + prow * 2) = make_float2(m_run[h], l_run[h]);
        }
    }
}

// Merge of split-KV partial results: one warp per (split item, row of the item).
//   m = max_s m_s;  out = sum_s 2^(m_s - m) O_s / sum_s 2^(m_s - m) l_s
struct MergeParams {
    const float* part_o;
    const float* part_ml;
    __nv_bfloat16* out;
    PlanDev plan;
    int N, Hq, Hkv, G, R, D, rows_per_item, items;
    int rows_used;     // min(rows_per_item, R): rows of an item that can exist
    long warps_total;  // split items * rows_used
    const int* bal_hdr;      // balanced plan: [0] = items to merge (known on the device only)
    const int4* bal_merge;   // balanced plan: (pair, first slot, slots) per pair to merge, else nullptr
    int bal_groups;          // balanced plan: groups of CTAs
    SeqTable seq;            // per-sequence plan (hdr == nullptr otherwise); the grid then covers every item
};

__global__ void __launch_bounds__(256, 4) attn_merge_kernel(MergeParams p) {
    const long w = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (w >= p.warps_total) return;
    const int lane = threadIdx.x & 31;
    const int k = (int)(w / p.rows_used), rloc = (int)(w % p.rows_used);
    // the k-th item that owns slots: group a comes first when it is split at all
    int item, nsplit, slot0;
    const int split_a = p.plan.splits_a > 1 ? p.plan.items_a : 0;
    if (p.bal_merge) {
        // the list of cut items was made on the device; the grid covers the most there can be
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const int tpu = p.plan.tiles_per_unit, rt = k % tpu;
        const int listed = p.bal_hdr[0];
        const int4 rec = p.bal_merge[k / tpu];       // a (sequence, kv head) pair that was cut (read beside the count)
        if (k / tpu >= listed) return;
        item = rec.x * tpu + rt; slot0 = rt * 2 * p.bal_groups + rec.y; nsplit = rec.z;
    } else if (p.seq.hdr) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const int per_seq = p.Hkv * p.plan.tiles_per_unit;
        const int b = k / per_seq;
        nsplit = p.seq.nsplit[b];
        if (nsplit == 1) return;                       // the item was stored by its only unit
        item = k;
        slot0 = p.seq.slot_off[b] + (k - b * per_seq) * nsplit;
    } else if (k < split_a) {
        item = k; nsplit = p.plan.splits_a; slot0 = k * p.plan.splits_a;
    } else {
        item = p.plan.items_a + (k - split_a); nsplit = p.plan.splits_b;
        slot0 = split_a * p.plan.splits_a + (k - split_a) * p.plan.splits_b;
    }
    const int unit = item / p.plan.tiles_per_unit;
    const int row = (item % p.plan.tiles_per_unit) * p.rows_per_item + rloc;
    if (row >= p.R) return;
    const int b = unit / p.Hkv, c = unit % p.Hkv;
    // Launched as a programmatic dependent of the attention kernel: the blocks may become
    // resident while that kernel drains; its partial results are only visible after this wait.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // A row costs one trip to memory when it has up to four parts (maxima, sums and accumulators
    // of all of them are fetched together), and two more per further group of four.
    const float* ml_base = p.part_ml + ((size_t)slot0 * p.rows_per_item + rloc) * 2;
    const size_t ml_stride = (size_t)p.rows_per_item * 2;
    const int per_lane = p.D / 32;  // 2 or 4 consecutive floats per lane
    const float* o_base = p.part_o + ((size_t)slot0 * p.rows_per_item + rloc) * p.D + lane * per_lane;
    const size_t o_stride = (size_t)p.rows_per_item * p.D;
    auto fetch = [&](int s0, float2 (&ml)[4], float4 (&v)[4]) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bool in = s0 + j < nsplit;
            ml[j] = in ? *reinterpret_cast<const float2*>(ml_base + (size_t)(s0 + j) * ml_stride)
                       : make_float2(-CUDART_INF_F, 0.f);
            const float* src = o_base + (size_t)(s0 + j) * o_stride;
            if (!in) v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            else if (per_lane == 4) v[j] = *reinterpret_cast<const float4*>(src);
            else { const float2 t = *reinterpret_cast<const float2*>(src); v[j] = make_float4(t.x, t.y, 0.f, 0.f); }
        }
    };
    float2 ml[4];
    float4 v[4];
    fetch(0, ml, v);
    float m = fmaxf(fmaxf(ml[0].x, ml[1].x), fmaxf(ml[2].x, ml[3].x));
#pragma unroll 1
    for (int s0 = 4; s0 < nsplit; s0 += 4) {
        float mv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) mv[j] = s0 + j < nsplit ? ml_base[(size_t)(s0 + j) * ml_stride] : -CUDART_INF_F;
#pragma unroll
        for (int j = 0; j < 4; ++j) m = fmaxf(m, mv[j]);
    }
    const float m_use = m == -CUDART_INF_F ? 0.f : m;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    float l = 0.f;
#pragma unroll 1
    for (int s0 = 0; s0 < nsplit; s0 += 4) {
        if (s0 > 0) fetch(s0, ml, v);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float wgt = exp2f(ml[j].x - m_use);     // 0 for an absent or empty split
            l += wgt * ml[j].y;
            acc[0] += wgt * v[j].x; acc[1] += wgt * v[j].y; acc[2] += wgt * v[j].z; acc[3] += wgt * v[j].w;
        }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    __nv_bfloat16* dst = p.out + (((size_t)b * p.N + row / p.G) * p.Hq + c * p.G + row % p.G) * p.D + lane * per_lane;
    if (per_lane == 4) {
        uint2 v;
        v.x = pack_bf16(acc[0] * inv, acc[1] * inv);
        v.y = pack_bf16(acc[2] * inv, acc[3] * inv);
        *reinterpret_cast<uint2*>(dst) = v;
    } else {
        *reinterpret_cast<uint32_t*>(dst) = pack_bf16(acc[0] * inv, acc[1] * inv);
    }
}

template <int D>
int launch_mma_t(const AttnArgs& a) {
    MmaParams p;
    p.q = (const __nv_bfloat16*)a.q; p.k_cache = (const __nv_bfloat16*)a.k_cache;
    p.v_cache = (const __nv_bfloat16*)a.v_cache; p.draft_k = (const __nv_bfloat16*)a.draft_k;
    p.draft_v = (const __nv_bfloat16*)a.draft_v; p.mask = a.mask; p.seq_lens = a.seq_lens;
    p.out = (__nv_bfloat16*)a.out; p.status = a.status;
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.Lmax = a.Lmax; p.G = a.G; p.W = a.W;
    p.R = a.N * a.G; p.scale_log2 = a.scale_log2; p.plan = a.plan.dev; p.slots = a.plan.slots;
    p.part_o = (float*)a.workspace;
    p.part_ml = (float*)((char*)a.workspace + plan_part_o_bytes(a.plan, a.D));
    const int smem = 4 * BN * D * 2;
    {
        static bool done[64] = {};   // per template instance: the opt-in sticks per device
        int dev = 0;
        GSD_CUDA_TRY(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64 || !done[dev]) {
            GSD_CUDA_TRY(cudaFuncSetAttribute(attn_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            if (dev >= 0 && dev < 64) done[dev] = true;
        }
    }
    dim3 grid(a.plan.ctas);
    attn_mma_kernel<D><<<grid, kThreads, smem, a.stream>>>(p);
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}

}  // namespace

int launch_attn_mma(const AttnArgs& a) {
    if (a.D == 128) return launch_mma_t<128>(a);
    if (a.D == 64) return launch_mma_t<64>(a);
    return GSD_ERR_BAD_SHAPE;
}

int launch_attn_merge(const AttnArgs& a) {
    MergeParams p;
    p.part_o = (const float*)a.workspace;
    p.part_ml = (const float*)((const char*)a.workspace + plan_part_o_bytes(a.plan, a.D));
    p.out = (__nv_bfloat16*)a.out;
    p.plan = a.plan.dev;
    p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.G = a.G; p.R = a.N * a.G; p.D = a.D;
    p.rows_per_item = a.plan.rows_per_item; p.items = a.plan.items;
    int split_items = (a.plan.dev.splits_a > 1 ? a.plan.dev.items_a : 0) +
                      (a.plan.dev.splits_b > 1 ? a.plan.items - a.plan.dev.items_a : 0);
    p.bal_hdr = nullptr;
    p.bal_merge = nullptr;
    p.bal_groups = 0;
    p.seq.hdr = nullptr; p.seq.nsplit = nullptr; p.seq.unit_off = nullptr; p.seq.slot_off = nullptr;
    if (a.plan.dev.balanced == 2) {
        p.seq = plan_seq_table(a.plan, a.D, a.B, a.workspace);
        split_items = a.plan.items;
    } else if (a.plan.dev.balanced) {
        const BalTable t = plan_bal_table(a.plan, a.D, a.workspace);
        p.bal_hdr = t.hdr;
        p.bal_merge = t.merge;
        const int tpu = a.plan.dev.tiles_per_unit, groups = a.plan.ctas / tpu, pairs = a.plan.items / tpu;
        p.bal_groups = groups;
        split_items = (pairs < groups - 1 ? pairs : groups - 1) * tpu;   // one pair per cut at most
    }
    p.rows_used = p.R < a.plan.rows_per_item ? p.R : a.plan.rows_per_item;
    p.warps_total = (long)split_items * p.rows_used;
    if (p.warps_total == 0) return GSD_OK;
    const int warps = 8;
    const long blocks = (p.warps_total + warps - 1) / warps;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(warps * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    GSD_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_merge_kernel, p));
    return GSD_OK;
}

}  // namespace gsd
