// Balanced work plan of gsd_verify_attn (tcgen05 back end), built on the device from seq_lens.
//
// Tree attention (Sec. 4.1) reads, per sequence, the committed prefix in the KV cache
// (Sec. 4.2) and the draft rows; the prefixes of a batch differ in length, and only the device
// knows by how much.  The key tiles of all (sequence, kv head) pairs are laid end to end on one
// line - pairs in index order, each with ceil(len/128) prefix tiles followed by all of its draft
// tiles - and group g of CTAs takes the g-th share of `share` tiles.  A group has one CTA per
// row-tile item of a pair: its CTAs walk the same key ranges at the same time, each for its own
// rows, so the K and V tiles are fetched from HBM once and shared through L2.  One block
// computes, for every group, the units that its share cuts out of the pairs, numbers the
// partial results along the line and lists the pairs that were cut (with their run of slots)
// for the merge pass.
#include "gsd_internal.cuh"

namespace gsd {
namespace {

constexpr int kPlanThreads = 1024;

struct PlanParams {
    const int32_t* seq_lens;
    int B, Lmax;
    int per_seq;      // (sequence, kv head) pairs per sequence = kv heads
    int nd;           // draft tiles per pair
    int ctas;         // groups of CTAs = shares
    BalTable t;
};

// exclusive prefix sum over the block; every thread also gets the total
__device__ unsigned long long block_scan(unsigned long long v, unsigned long long* s_warp, unsigned long long* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();                       // s_warp may still be read from an earlier scan
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        unsigned long long w = s_warp[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, w, o);
            if (lane >= o) w += t;
        }
        s_warp[lane] = w;                  // inclusive over warps
    }
    __syncthreads();
    *total = s_warp[31];
    return inc - v + (warp ? s_warp[warp - 1] : 0ull);
}

constexpr int kPlanSeqsOnChip = 4096;   // sequences whose line offsets are kept in shared memory

__global__ void __launch_bounds__(kPlanThreads) attn_plan_kernel(PlanParams p) {
    __shared__ unsigned long long s_warp[32];
    __shared__ int s_off[kPlanSeqsOnChip + 1];
    __shared__ int s_tiles[kPlanSeqsOnChip];
    const int tid = threadIdx.x;
    // the attention kernel may set itself up meanwhile; it waits before it reads the table
    if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const bool on_chip = p.B <= kPlanSeqsOnChip;
    auto tiles_of = [&](int b) -> int {
        int L = p.seq_lens[b];
        L = L < 0 ? 0 : (L > p.Lmax ? p.Lmax : L);
        return (L + 127) / 128 + p.nd;
    };
    // 1. where each sequence starts on the line
    const int chunk = (p.B + kPlanThreads - 1) / kPlanThreads;
    const int b_lo = min(tid * chunk, p.B), b_hi = min(b_lo + chunk, p.B);
    unsigned long long mine = 0;
    for (int b = b_lo; b < b_hi; ++b) mine += (unsigned long long)p.per_seq * tiles_of(b);
    unsigned long long total64;
    unsigned long long run = block_scan(mine, s_warp, &total64);
    for (int b = b_lo; b < b_hi; ++b) {
        const int T = tiles_of(b);
        p.t.off[b] = (int)run;
        if (on_chip) { s_off[b] = (int)run; s_tiles[b] = T; }
        run += (unsigned long long)p.per_seq * T;
    }
    const int total = (int)total64;        // (the host keeps the line below 2^30 tiles)
    if (tid == 0) {
        p.t.off[p.B] = total;
        if (on_chip) s_off[p.B] = total;
    }
    __syncthreads();
    const int* off = on_chip ? s_off : p.t.off;
    auto tiles_at = [&](int b) -> int { return on_chip ? s_tiles[b] : (off[b + 1] - off[b]) / p.per_seq; };

    // 2. the share of group `tid`
    const int share = max(1, (total + p.ctas - 1) / p.ctas);
    const bool active = tid < p.ctas;
    const long long a64 = (long long)tid * share;
    const int a = active ? (int)min(a64, (long long)total) : total;
    const int e = min(a + share, total);
    // the pair that holds a position of the line: (sequence, pair inside it, its tile range)
    struct At { int b, ci, lo, hi; };
    auto locate = [&](int pos) -> At {
        int lo = 0, hi = p.B - 1;          // the last b with off[b] <= pos
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (off[mid] <= pos) lo = mid; else hi = mid - 1;
        }
        At r;
        r.b = lo;
        const int T = tiles_at(lo);
        r.ci = (pos - off[lo]) / T;
        r.lo = off[lo] + r.ci * T;
        r.hi = r.lo + T;
        return r;
    };
    // how many units and partial results the share [a, e) makes: from its two ends alone
    int n_units = 0, n_partial = 0;
    At first = {0, 0, 0, 0};
    if (a < e) {
        first = locate(a);
        const At last = locate(e - 1);
        n_units = (last.b * p.per_seq + last.ci) - (first.b * p.per_seq + first.ci) + 1;
        n_partial = n_units == 1 ? ((a > first.lo || e < first.hi) ? 1 : 0)
                                 : (a > first.lo ? 1 : 0) + (e < last.hi ? 1 : 0);
    }
    // a pair is listed for the merge pass by the group whose share starts at the first cut inside it
    const bool cut_here = a < e && a > first.lo;
    const bool first_cut = cut_here && (a64 - share <= (long long)first.lo);
    const unsigned long long packed = (unsigned long long)n_units | ((unsigned long long)n_partial << 32) |
                                      ((unsigned long long)(first_cut ? 1 : 0) << 48);
    unsigned long long tot;
    const unsigned long long ex = block_scan(packed, s_warp, &tot);
    const int ubase = (int)(ex & 0xFFFFFFFFull);
    const int sbase = (int)((ex >> 32) & 0xFFFFull);
    const int mbase = (int)(ex >> 48);
    if (active) {
        // walk over the pairs that the share touches and write its units
        int pos = a, b = first.b, n = 0, q = 0;
        while (pos < e) {
            while (pos >= off[b + 1]) ++b;
            const int T = tiles_at(b);
            const int ci = (pos - off[b]) / T;
            const int lo = off[b] + ci * T, hi = lo + T;
            const int t0 = pos - lo, t1 = min(e, hi) - lo;
            const bool partial = t0 > 0 || t1 < T;
            p.t.units[ubase + n] = make_int4(b * p.per_seq + ci, t0, t1, partial ? sbase + q : -1);
            ++n;
            q += partial ? 1 : 0;
            pos = lo + t1;
        }
        p.t.cta[tid] = make_int2(ubase, n_units);
        if (first_cut) {
            // cuts inside the pair: a, a + share, ... below its end
            const int cuts = (first.hi - 1 - a) / share + 1;
            p.t.merge[mbase] = make_int4(first.b * p.per_seq + first.ci, sbase - 1, cuts + 1, 0);
        }
    }
    if (tid == 0) {
        p.t.hdr[0] = (int)(tot >> 48);
        p.t.hdr[1] = total;
        p.t.hdr[2] = share;
    }
}

struct SeqPlanParams {
    const int32_t* seq_lens;
    int B, Lmax;
    int per_seq;        // work items per sequence (kv heads x row-tile items)
    int nd;             // draft tiles per item
    int units_wanted;
    int slots_cap;      // partial-result slots the workspace holds
    SeqTable t;
};

// Per-sequence split counts: one block, sequences dealt out in contiguous chunks to its threads.
__global__ void __launch_bounds__(kPlanThreads) attn_plan_seq_kernel(SeqPlanParams p) {
    __shared__ unsigned long long s_warp[32];
    const int tid = threadIdx.x;
    if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    auto tiles_of = [&](int b) -> int {
        int L = p.seq_lens[b];
        L = L < 0 ? 0 : (L > p.Lmax ? p.Lmax : L);
        return (L + 127) / 128 + p.nd;
    };
    const int chunk = (p.B + kPlanThreads - 1) / kPlanThreads;
    const int b_lo = min(tid * chunk, p.B), b_hi = min(b_lo + chunk, p.B);
    unsigned long long mine = 0;
    for (int b = b_lo; b < b_hi; ++b) mine += (unsigned long long)p.per_seq * tiles_of(b);
    unsigned long long total64;
    block_scan(mine, s_warp, &total64);
    // the common target length of a unit: at least four key tiles
    const long long target64 = (long long)((total64 + p.units_wanted - 1) / p.units_wanted);
    const int target = (int)(target64 < 4 ? 4 : (target64 > (1 << 30) ? (1 << 30) : target64));
    auto splits_of = [&](int b) -> int {
        const int n = (2 * tiles_of(b) + target) / (2 * target);      // tiles / target, rounded
        return n < 1 ? 1 : (n > kSeqPlanMaxSplit ? kSeqPlanMaxSplit : n);
    };
    unsigned long long units = 0, slots = 0;
    for (int b = b_lo; b < b_hi; ++b) {
        const int n = splits_of(b);
        units += (unsigned long long)n * p.per_seq;
        if (n > 1) slots += (unsigned long long)n * p.per_seq;
    }
    // (both sums stay far below 2^31: at most 32 x items each)
    unsigned long long tot;
    const unsigned long long ex = block_scan(units | (slots << 32), s_warp, &tot);
    // should the partial results not fit the workspace (the host's bound makes sure they do),
    // nothing is cut at all
    const bool fits = (tot >> 32) <= (unsigned long long)p.slots_cap;
    unsigned long long u = ex & 0xFFFFFFFFull, sl = ex >> 32;
    for (int b = b_lo; b < b_hi; ++b) {
        const int n = fits ? splits_of(b) : 1;
        p.t.nsplit[b] = n;
        p.t.unit_off[b] = fits ? (int)u : b * p.per_seq;
        p.t.slot_off[b] = fits ? (int)sl : 0;
        u += (unsigned long long)n * p.per_seq;
        if (n > 1) sl += (unsigned long long)n * p.per_seq;
    }
    if (tid == 0) {
        const int total_units = fits ? (int)(tot & 0xFFFFFFFFull) : p.B * p.per_seq;
        p.t.unit_off[p.B] = total_units;
        p.t.slot_off[p.B] = fits ? (int)(tot >> 32) : 0;
        p.t.hdr[0] = total_units;
        p.t.hdr[1] = (int)(total64 > 0x7FFFFFFFull ? 0x7FFFFFFFull : total64);
        p.t.hdr[2] = target;
    }
}

}  // namespace

int launch_attn_plan(const AttnArgs& a) {
    if (!a.plan.dev.balanced) return GSD_OK;
    if (a.plan.dev.balanced == 2) {
        SeqPlanParams p;
        p.seq_lens = a.seq_lens;
        p.B = a.B; p.Lmax = a.Lmax;
        p.per_seq = a.Hkv * a.plan.dev.tiles_per_unit;
        p.nd = (a.N + 127) / 128;
        p.units_wanted = kSeqPlanWaves * a.plan.ctas;
        p.slots_cap = a.plan.slots;
        p.t = plan_seq_table(a.plan, a.D, a.B, a.workspace);
        attn_plan_seq_kernel<<<1, kPlanThreads, 0, a.stream>>>(p);
        GSD_CUDA_TRY(cudaGetLastError());
        return GSD_OK;
    }
    if (a.plan.ctas / a.plan.dev.tiles_per_unit > kPlanThreads) return GSD_ERR_BAD_SHAPE;
    PlanParams p;
    p.seq_lens = a.seq_lens;
    p.B = a.B; p.Lmax = a.Lmax;
    p.per_seq = a.Hkv;
    p.nd = (a.N + 127) / 128;
    p.ctas = a.plan.ctas / a.plan.dev.tiles_per_unit;
    p.t = plan_bal_table(a.plan, a.D, a.workspace);
    attn_plan_kernel<<<1, kPlanThreads, 0, a.stream>>>(p);
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}

}  // namespace gsd
