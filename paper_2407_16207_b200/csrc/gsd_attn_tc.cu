// gsd_verify_attn, tcgen05 back end for D = 128 (sm_100a): TMA-fed, TMEM-resident
// flash-attention over the stacked (draft node x GQA head) rows.
//
// Tree attention over the flattened token graph (Sec. 4.1) with the committed prefix in the
// KV cache (Sec. 4.2): row r = (node r / G, head r % G) of kv head c attends to cache rows
// j < seq_lens[b] and to the draft rows whose bit is set in the node's ancestor mask.
//
// A unit of work is up to two row tiles of 128 stacked rows of one (sequence, kv head) and a
// contiguous range of 128-key tiles (prefix tiles, then the draft tiles that hold a visible
// key for any of its rows).  Warp roles:
//   warps 0-3   softmax of stream 0 (thread = row = TMEM lane)
//   warps 4-7   softmax of stream 1
//   warp  8     TMA producer (one thread): Q once, then K and V tiles into two smem rings
//   warp  9     QK^T issuer, warp 11 PV issuer (converged, one elected lane per instruction)
//   warp 10     TMEM allocation / release
// A stream is a row tile (two row tiles: both streams see every key tile) or, for a unit with
// one row tile, the even / odd key tiles of that row tile (merged in the epilogue).  A job is
// one key tile of one stream; jobs alternate between the streams.
// TMEM (512 columns): S (128) | P0 (64) | P1 (64) | O0 (128) | O1 (128).  There is one score
// buffer: QK^T of job k+1 is issued as soon as the softmax of job k has pulled its score row
// into registers, i.e. it runs under that softmax; P (bf16) has a buffer per stream and
// O_i += P_i V follows when the softmax hands P over (in two halves of 64 keys).  So neither
// softmax warpgroup ever waits for a QK^T that could not start.  The two kinds of MMA are
// issued by two warps on different schedulers, each paced only by its own barriers (the
// softmax warps are almost always ready to issue, so one issuing warp gets too few slots
// to feed the tensor pipe).  The running maximum is only raised when a tile
// exceeds it by more than 2^8 (the accumulator rescale is then done in place in TMEM by the
// row's own thread), so P <= 256 and the rescale is rare.  Every mbarrier wait is bounded: on
// expiry the kernel raises GSD_DEV_WAIT_EXPIRED, all roles leave their loops, TMEM is released.
#include "gsd_internal.cuh"
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>
#include <stdio.h>

namespace gsd {
namespace {

constexpr int BM = 128;            // rows per row tile
constexpr int BN = 128;            // keys per tile
constexpr int HD = 128;            // head dimension
constexpr int KST = 2;             // K ring stages
constexpr int VST = 2;             // V ring stages
constexpr uint32_t HALF_BYTES = 128 * 64 * 2;     // one [128 rows][64 bf16] swizzled block
constexpr uint32_t TILE_BYTES = 2 * HALF_BYTES;   // a 128 x 128 bf16 tile (two column halves)
constexpr int kThreads = 384;
constexpr uint32_t kSmemBytes = (2 + KST + VST) * TILE_BYTES + 2 * HALF_BYTES + 1024;  // tiles, output staging, alignment slack
constexpr float kRescaleThreshold = 8.0f;         // log2 units
constexpr int kUnitTable = 12;                    // units of work per CTA decoded in the prologue (one per warp)
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // default limit of every in-kernel wait

// Test hook (see gsd_debug_attn_wait): a shorter limit and, optionally, a CTA's first K tile
// withheld so that a wait really runs out.
unsigned long long g_wait_limit_ns = kWaitLimitNs;
int g_withhold_first_k = 0;

// What every bounded wait looks at, in shared memory: word 0 is raised by the first wait that
// gives up (all other waits then return within a few polls), words 2-3 hold the time limit.
struct WaitCtl {
    int abort;
    int pad;
    unsigned long long limit_ns;
};

// TMEM columns (32-bit words): one score tile, a bf16 P tile per stream, an accumulator per stream
constexpr uint32_t COL_S = 0, COL_P0 = 128, COL_P1 = 192, COL_O0 = 256, COL_O1 = 384;

enum Bar {
    BAR_Q_FULL = 0,
    BAR_K_FULL = 1,                   // KST
    BAR_K_EMPTY = BAR_K_FULL + KST,   // KST
    BAR_V_FULL = BAR_K_EMPTY + KST,   // VST
    BAR_V_EMPTY = BAR_V_FULL + VST,   // VST
    BAR_S_FULL = BAR_V_EMPTY + VST,   // 2: the scores of a job of stream i are in S
    BAR_S_FREE = BAR_S_FULL + 2,      // 2: the softmax of stream i has read them out of S
    BAR_P_READY = BAR_S_FREE + 2,     // 2: keys 0..63 of P_i are in TMEM
    BAR_P_READY2 = BAR_P_READY + 2,   // 2: keys 64..127 of P_i are in TMEM
    BAR_P_FREE = BAR_P_READY2 + 2,    // 2: the PV of a job of stream i (and all before it) has completed
    BAR_O_DONE = BAR_P_FREE + 2,      // 2: every PV of the unit on stream i has completed
    BAR_O_FREE = BAR_O_DONE + 2,      // 2: the accumulator rows of the unit have been read out
    BAR_Q_EMPTY = BAR_O_FREE + 2,     // 1: every QK^T of the unit has completed
    BAR_ML_READY = BAR_Q_EMPTY + 1,   // 1: (max, sum) of the odd-tile stream are in shared memory
    BAR_DRAIN = BAR_ML_READY + 1,     // 2: every MMA issued by the QK^T / PV warp has completed
    BAR_COUNT = BAR_DRAIN + 2
};

struct TcParams {
    const uint32_t* mask;
    const int32_t* seq_lens;
    __nv_bfloat16* out;
    float* part_o;
    float* part_ml;
    int32_t* status;
    int B, N, Hq, Hkv, Lmax, G, W, R;
    float scale_log2;
    PlanDev plan;
    int total_work;   // CTAs of the plan = units of work
    int slots;        // partial-result slots of the plan
    const int2* bal_cta;     // balanced plan: (first unit, units) of every group of CTAs, else nullptr
    const int4* bal_units;   // balanced plan: (pair, first tile, end tile, slot or -1)
    SeqTable seq;            // per-sequence plan: split counts and unit / slot offsets (hdr == nullptr otherwise)
    unsigned long long wait_limit_ns;
    int withhold_first_k;   // test hook: every CTA leaves out the K copy of its first key tile
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false when the wait gave up (time limit, or another role raised the
// abort flag); the caller then leaves its loop.  `ignore_abort` is for the final drain.
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            int32_t* status, bool ignore_abort) {
    const unsigned long long t0 = global_ns();
    const unsigned long long limit = reinterpret_cast<const volatile WaitCtl*>(abort_flag)->limit_ns;
    for (unsigned it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (!ignore_abort && *abort_flag) return false;
            if (global_ns() - t0 > limit) {
                *abort_flag = 1;
                if (status) atomicOr((unsigned*)status, GSD_DEV_WAIT_EXPIRED);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status, false);
}
// the same, called by all lanes of a converged warp; the answer is made uniform
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               int32_t* status) {
    return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort_flag, status));
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// shared -> global tile store; completion is tracked by bulk async-groups of the issuing thread
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
        ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void wg_barrier(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }
// the same hardware barrier of a warpgroup with an AND over a flag: every thread gets the answer
__device__ __forceinline__ bool wg_all(int id, bool flag) {
    uint32_t r;
    asm volatile(
        "{\n .reg .pred p, q;\n setp.ne.u32 q, %2, 0;\n bar.red.and.pred p, %1, 128, q;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(r) : "r"(id), "r"((uint32_t)flag) : "memory");
    return r != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// The MMA warp runs its loops with all 32 lanes converged and elects one lane per tcgen05
// instruction: addresses, descriptors and loop state are then warp-uniform, which costs the
// warp far fewer issue slots than a single-lane branch would (the softmax warps on the same
// scheduler are almost always ready to issue, so every extra instruction here waits its turn).
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile(
        "{\n .reg .pred q;\n elect.sync _|q, 0xffffffff;\n"
        " @q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}\n" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread t of the warp gets lane (base + t)
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const float (&v)[32]) {
    const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// pointer form: v[0..31] must be register-resident (constant indices after unrolling)
__device__ __forceinline__ void tc_ld32p(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// packed fp32 pairs (one instruction for two lanes of arithmetic)
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d)
        : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)),
          "l"(*reinterpret_cast<unsigned long long*>(&c)));
    return *reinterpret_cast<float2*>(&d);
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d)
        : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)));
    return *reinterpret_cast<float2*>(&d);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// ---- shared-memory matrix descriptors (128-byte swizzle, 8-row groups 1024 bytes apart)
constexpr uint64_t kDescBase = (1ull << 46) | (2ull << 61);   // descriptor version 1, SWIZZLE_128B
// K-major operand (rows x 64 bf16 per block): leading offset unused (1), stride = 1024 B.
// MN-major operand (V: [key][64 d] blocks): leading offset = distance between the two
// 64-column blocks, stride = 1024 B between 8-key groups.
// Descriptors are handled as (low word, high word): the high word is common to both kinds, and
// a k-step only adds a small constant to the start-address field of the low word (the
// tiles sit below 256 KB, so the sum stays inside the 14-bit field).
constexpr uint32_t kDescHi = (uint32_t)((kDescBase | ((uint64_t)(1024 >> 4) << 32)) >> 32);
__device__ __forceinline__ uint32_t desc_lo_kmajor(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ uint32_t desc_lo_mnmajor(uint32_t addr) { return ((addr & 0x3FFFFu) >> 4) | ((HALF_BYTES >> 4) << 16); }
// instruction descriptors: bf16 x bf16 -> fp32, M = 128, N = 128
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescPV = kIdescQK | (1u << 16);   // B (= V) is MN-major

// S = A B^T over the head dimension (eight k-steps of 16) as one block issued by one elected
// lane: per k-step one add per operand and the MMA, nothing else.  alo / blo are the low
// descriptor words of two K-major [128][128] bf16 tiles (two swizzled 64-column blocks each).
__device__ __forceinline__ void tc_qk8(uint32_t d_tmem, uint32_t alo, uint32_t blo) {
#define GSD_QK_STEP(OFF, P)                                                         \
    " add.u32 al, %1, " #OFF ";\n add.u32 bl, %2, " #OFF ";\n"                       \
    " mov.b64 a, {al, %3};\n mov.b64 b, {bl, %3};\n"                                \
    " @q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %4, " #P ";\n"
    asm volatile(
        "{\n .reg .pred q, pt, pf;\n .reg .b64 a, b;\n .reg .b32 al, bl;\n"
        " elect.sync _|q, 0xffffffff;\n"
        " setp.eq.u32 pt, %4, %4;\n setp.ne.u32 pf, %4, %4;\n"
        GSD_QK_STEP(0, pf) GSD_QK_STEP(2, pt) GSD_QK_STEP(4, pt) GSD_QK_STEP(6, pt)
        GSD_QK_STEP(1024, pt) GSD_QK_STEP(1026, pt) GSD_QK_STEP(1028, pt) GSD_QK_STEP(1030, pt)
        "}\n"
        ::"r"(d_tmem), "r"(alo), "r"(blo), "r"(kDescHi), "r"(kIdescQK) : "memory");
#undef GSD_QK_STEP
}
// O (+)= P V for four k-steps of 16 keys: A = 8 TMEM columns of bf16 pairs per step, B = the
// MN-major V tile (2048 bytes per 16 keys).  `accum_first` = 0 makes the first step overwrite O.
__device__ __forceinline__ void tc_pv4(uint32_t d_tmem, uint32_t a_tmem, uint32_t blo, uint32_t accum_first) {
#define GSD_PV_STEP(ACOL, BOFF, P)                                                  \
    " add.u32 at, %1, " #ACOL ";\n add.u32 bl, %2, " #BOFF ";\n mov.b64 b, {bl, %3};\n" \
    " @q tcgen05.mma.cta_group::1.kind::f16 [%0], [at], b, %4, " #P ";\n"
    asm volatile(
        "{\n .reg .pred q, pt, p0;\n .reg .b64 b;\n .reg .b32 at, bl;\n"
        " elect.sync _|q, 0xffffffff;\n"
        " setp.eq.u32 pt, %4, %4;\n setp.ne.u32 p0, %5, 0;\n"
        GSD_PV_STEP(0, 0, p0) GSD_PV_STEP(8, 128, pt) GSD_PV_STEP(16, 256, pt) GSD_PV_STEP(24, 384, pt)
        "}\n"
        ::"r"(d_tmem), "r"(a_tmem), "r"(blo), "r"(kDescHi), "r"(kIdescPV), "r"(accum_first) : "memory");
#undef GSD_PV_STEP
}


struct TileInfo {
    int kind;     // 0 full prefix tile, 1 ragged prefix tile, 2 draft tile
    int key0;     // first key (prefix position or draft node) of the tile; negative for a ragged tile of a prefix below 128
    int nvalid;   // prefix: visible keys in the tile (the last nvalid of a ragged tile)
};

__device__ __forceinline__ TileInfo tile_info(int t, int nPT, int L, unsigned live) {
    TileInfo ti;
    if (t < nPT) {
        ti.key0 = t * BN;
        ti.nvalid = min(BN, L - ti.key0);
        ti.kind = ti.nvalid == BN ? 0 : 1;
        // The ragged last tile is loaded as the LAST 128 rows of the prefix (rows before position
        // 0 are filled with zeros by the copy engine): it then holds no row past the sequence
        // end, whose contents could be anything, and its first 128 - nvalid keys, which the tile
        // before it has covered already, are masked like invisible draft keys.
        if (ti.kind == 1) ti.key0 = L - BN;
    } else {
        int k = t - nPT, d = 0;
        for (;; ++d) {   // the k-th set bit of `live`
            if ((live >> d) & 1u) {
                if (k == 0) break;
                --k;
            }
        }
        ti.key0 = d * BN;
        ti.nvalid = BN;
        ti.kind = 2;
    }
    return ti;
}

// What a role needs to know about one unit of work (a row pair of one (sequence, kv head) and
// a key range).  Every warp derives it on its own from the work index, so the roles never
// have to meet at a CTA-wide barrier between units.
struct UnitInfo {
    int b, c, row0, split, nsplit, slot;
    int L, nPT, t_begin, ntiles;
    unsigned live;   // draft tiles (128 nodes each) holding a visible key for any row of the unit
    bool two;        // the second row tile exists
};

// `w` is the work index of a fixed plan, or the index of the group's unit in the table of a balanced one.
__device__ __forceinline__ UnitInfo unit_info(const TcParams& p, int w, int lane) {
    UnitInfo u;
    int item, t0n = 0, t1n = 0;
    const bool bal = p.bal_units != nullptr;
    if (bal) {
        // the unit of this CTA's group, for the row-tile item this CTA has in every pair
        const int tpu = p.plan.tiles_per_unit, rt = (int)blockIdx.x % tpu;
        const int4 rec = p.bal_units[w];
        item = rec.x * tpu + rt; t0n = rec.y; t1n = rec.z;
        u.slot = rec.w >= 0 ? rt * 2 * ((int)gridDim.x / tpu) + rec.w : -1;
        u.split = 0;
        u.nsplit = rec.w >= 0 ? 2 : 1;     // only "one piece or several" matters below
    } else if (p.seq.hdr) {
        // unit w of the per-sequence plan: the last sequence whose first unit is <= w, then
        // (key range, item) inside it
        int lo = 0, hi = p.B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (p.seq.unit_off[mid] <= w) lo = mid; else hi = mid - 1;
        }
        const int per_seq = p.Hkv * p.plan.tiles_per_unit;
        const int r = w - p.seq.unit_off[lo];
        u.nsplit = p.seq.nsplit[lo];
        u.split = r / per_seq;
        const int i = r - u.split * per_seq;
        item = lo * per_seq + i;
        u.slot = u.nsplit > 1 ? p.seq.slot_off[lo] + i * u.nsplit + u.split : 0;
    } else {
        plan_decode(p.plan, w, item, u.split, u.nsplit, u.slot);
    }
    const int unit = item / p.plan.tiles_per_unit;
    u.row0 = (item % p.plan.tiles_per_unit) * (2 * BM);
    u.b = unit / p.Hkv;
    u.c = unit % p.Hkv;
    u.two = u.row0 + BM < p.R;
    if (!GSD_IN_BOUNDS(u.b >= 0 && u.b < p.B && u.c < p.Hkv && u.row0 < p.R, p.status)) {
        u.b = 0; u.c = 0; u.row0 = 0; u.two = false;      // checking build only: a unit outside the problem
    }
    int L = p.seq_lens[u.b];
    L = L < 0 ? 0 : (L > p.Lmax ? p.Lmax : L);
    u.L = L;
    // OR the mask rows of the unit's nodes, one node per lane
    const int n_lo = u.row0 / p.G;
    const int n_hi = (min(u.row0 + 2 * BM, p.R) - 1) / p.G + 1;
    unsigned live = 0;
    const uint32_t tail = (p.N & 31) ? (1u << (p.N & 31)) - 1u : 0xFFFFFFFFu;   // valid bits of the last word
    if ((p.W & 3) == 0 && (reinterpret_cast<uintptr_t>(p.mask) & 15u) == 0) {
        // four words = one draft tile per 16-byte load; all loads of a row are issued before any is used
        for (int n = n_lo + lane; n < n_hi; n += 32) {
            const uint4* mrow = reinterpret_cast<const uint4*>(p.mask + ((size_t)u.b * p.N + n) * p.W);
            uint4 q[GSD_MAX_NODES / 128];
#pragma unroll
            for (int t = 0; t < GSD_MAX_NODES / 128; ++t) q[t] = t < (p.W >> 2) ? mrow[t] : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int t = 0; t < GSD_MAX_NODES / 128; ++t) {
                if (t == (p.W >> 2) - 1) q[t].w &= tail;
                if (q[t].x | q[t].y | q[t].z | q[t].w) live |= 1u << t;
            }
        }
    } else {
        for (int n = n_lo + lane; n < n_hi; n += 32) {
            const uint32_t* mrow = p.mask + ((size_t)u.b * p.N + n) * p.W;
            for (int wi = 0; wi < p.W; ++wi) {
                uint32_t word = mrow[wi];
                if (wi == p.W - 1) word &= tail;
                if (word) live |= 1u << (wi >> 2);
            }
        }
    }
    u.live = __reduce_or_sync(0xFFFFFFFFu, live);
    u.nPT = (L + BN - 1) / BN;
    if (bal) {
        // the table counts every draft tile; here only those with a visible key are numbered
        auto live_index = [&](int t) { return t <= u.nPT ? t : u.nPT + __popc(u.live & ((1u << (t - u.nPT)) - 1u)); };
        u.t_begin = live_index(t0n);
        u.ntiles = live_index(t1n) - u.t_begin;
        return u;
    }
    const int T = u.nPT + __popc(u.live);
    const int per = (T + u.nsplit - 1) / u.nsplit;
    u.t_begin = min(u.split * per, T);
    u.ntiles = min(u.t_begin + per, T) - u.t_begin;
    return u;
}

// Persistent kernel: CTA k walks the work indices k, k + gridDim.x, ...  Barrier phases are
// counted across units, so the producer and the QK^T issuer run ahead into the next unit
// (Q, the first K/V tiles and the first QK^T) while the softmax warps still read out the
// accumulators of the previous one.
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_dk,
               const __grid_constant__ CUtensorMap tm_dv, const __grid_constant__ CUtensorMap tm_out,
               const TcParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bars[BAR_COUNT];
    __shared__ uint32_t s_tmem_base;
    __shared__ __align__(8) WaitCtl s_wait;
    __shared__ float2 s_ml1[BM];      // (max, sum) of the odd-tile stream, one per row
    __shared__ UnitInfo s_units[kUnitTable];   // the CTA's first units of work, decoded once up front

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = p.N, G = p.G, R = p.R;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;                                   // 2 tiles
    const uint32_t sK = smem_base + 2 * TILE_BYTES;                  // KST tiles
    const uint32_t sV = sK + KST * TILE_BYTES;                       // VST tiles
    const uint32_t sStage = sV + VST * TILE_BYTES;                   // one [128][64] bf16 block per softmax warpgroup
    const uint32_t bar0 = smem_u32(s_bars);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int* abort_flag = &s_wait.abort;

    if (tid == 0) {
        // the merge pass (a programmatic dependent launch) may be made resident as CTAs retire
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        s_wait.abort = 0;
        s_wait.limit_ns = p.wait_limit_ns;
        mbar_init(bar(BAR_Q_FULL), 1);
        mbar_init(bar(BAR_Q_EMPTY), 1);
        mbar_init(bar(BAR_ML_READY), 4);
        for (int s = 0; s < KST; ++s) { mbar_init(bar(BAR_K_FULL + s), 1); mbar_init(bar(BAR_K_EMPTY + s), 1); }
        for (int s = 0; s < VST; ++s) { mbar_init(bar(BAR_V_FULL + s), 1); mbar_init(bar(BAR_V_EMPTY + s), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(BAR_S_FULL + i), 1);
            mbar_init(bar(BAR_S_FREE + i), 4);     // one arrival per softmax warp
            mbar_init(bar(BAR_P_READY + i), 4);
            mbar_init(bar(BAR_P_READY2 + i), 4);
            mbar_init(bar(BAR_P_FREE + i), 1);
            mbar_init(bar(BAR_O_DONE + i), 1);
            mbar_init(bar(BAR_O_FREE + i), 4);
            mbar_init(bar(BAR_DRAIN + i), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 10) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&s_tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // The CTA's units: work indices blockIdx.x, blockIdx.x + gridDim.x, ... of a fixed plan, or
    // a run of the table that the planning kernel (this kernel is its programmatic dependent)
    // has written.
    int n_my;
    if (p.bal_cta) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        n_my = p.bal_cta[blockIdx.x / p.plan.tiles_per_unit].y;
    } else if (p.seq.hdr) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const int units = p.seq.hdr[0];
        n_my = units > (int)blockIdx.x ? (units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    } else {
        n_my = p.total_work > (int)blockIdx.x ? (p.total_work - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    }
    // (recomputed where it is needed rather than kept in a register through the key loops)
    auto unit_index = [&](int it) -> int {
        return p.bal_cta ? p.bal_cta[blockIdx.x / p.plan.tiles_per_unit].x + it : (int)blockIdx.x + it * (int)gridDim.x;
    };
    // Decoding a unit costs two dependent trips to global memory (sequence length, mask rows).
    // Each warp decodes one of the CTA's first units here, all at once, so that no role pays
    // that latency between units.
    for (int k = warp; k < kUnitTable; k += kThreads / 32) {
        if (k < n_my) {
            const UnitInfo u = unit_info(p, unit_index(k), lane);
            if (lane == 0) s_units[k] = u;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    auto unit_of = [&](int it) -> UnitInfo {
        return it < kUnitTable ? s_units[it] : unit_info(p, unit_index(it), lane);
    };

    if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 96;");
    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        int kvc = 0;          // key tiles loaded so far (ring position)
        int au = 0;           // non-empty units so far
        bool ok = true, q_pending = false;
        for (int it = 0; it < n_my && ok; ++it) {
            const UnitInfo u = unit_of(it);
            if (u.ntiles == 0) continue;
            if (lane == 0) {
                // Q of the previous unit is free once its last QK^T has completed
                ok = mbar_wait(bar(BAR_Q_EMPTY), (au & 1) ^ 1, abort_flag, p.status);
                if (ok) {
                    const int ntile_rows = u.two ? 2 : 1;
                    mbar_expect_tx(bar(BAR_Q_FULL), (uint32_t)ntile_rows * TILE_BYTES);
                    for (int i = 0; i < ntile_rows; ++i)
                        for (int h = 0; h < 2; ++h)
                            tma_load_4d(sQ + i * TILE_BYTES + h * HALF_BYTES, &tm_q, bar(BAR_Q_FULL), h * 64, u.c * G,
                                        (u.row0 + i * BM) / G, u.b);
                    q_pending = true;
                }
                for (int idx = 0; idx < u.ntiles && ok; ++idx) {
                    const TileInfo ti = tile_info(u.t_begin + idx, u.nPT, u.L, u.live);
                    const CUtensorMap* mk = ti.kind == 2 ? &tm_dk : &tm_k;
                    const CUtensorMap* mv = ti.kind == 2 ? &tm_dv : &tm_v;
                    const int s = kvc % KST;
                    const uint32_t par = (uint32_t)((kvc / KST) & 1) ^ 1u;
                    ok = mbar_wait(bar(BAR_K_EMPTY + s), par, abort_flag, p.status);
                    if (!ok) break;
                    mbar_expect_tx(bar(BAR_K_FULL + s), TILE_BYTES);
                    if (!(p.withhold_first_k && kvc == 0))   // (test hook: the bytes announced above never arrive)
                        for (int h = 0; h < 2; ++h)
                            tma_load_4d(sK + s * TILE_BYTES + h * HALF_BYTES, mk, bar(BAR_K_FULL + s), h * 64, u.c, ti.key0, u.b);
                    ok = mbar_wait(bar(BAR_V_EMPTY + s), par, abort_flag, p.status);
                    if (!ok) {
                        // the K copy just issued is still in flight: let it land
                        mbar_wait_slow(bar(BAR_K_FULL + s), (kvc / KST) & 1, abort_flag, nullptr, true);
                        break;
                    }
                    mbar_expect_tx(bar(BAR_V_FULL + s), TILE_BYTES);
                    for (int h = 0; h < 2; ++h)
                        tma_load_4d(sV + s * TILE_BYTES + h * HALF_BYTES, mv, bar(BAR_V_FULL + s), h * 64, u.c, ti.key0, u.b);
                    ++kvc;
                }
                if (!ok) {
                    // gave up: let the copies already in flight land before the CTA retires
                    if (q_pending) mbar_wait_slow(bar(BAR_Q_FULL), au & 1, abort_flag, nullptr, true);
                    for (int t = max(0, kvc - KST); t < kvc; ++t) {
                        mbar_wait_slow(bar(BAR_K_FULL + t % KST), (t / KST) & 1, abort_flag, nullptr, true);
                        mbar_wait_slow(bar(BAR_V_FULL + t % VST), (t / VST) & 1, abort_flag, nullptr, true);
                    }
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
            kvc = __shfl_sync(0xFFFFFFFFu, kvc, 0);
            ++au;
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------ QK^T issuer (all lanes converged)
        // S = Q K^T job by job.  Nothing orders these MMAs against the PV MMAs of warp 11 in the
        // tensor pipe, and nothing has to: they touch different TMEM columns, and every
        // hand-over (S to the softmax, P to the PV, S back) goes through an mbarrier.
        int kvc = 0;              // key tiles of earlier units (ring position of this unit's first tile)
        int au = 0;               // non-empty units so far
        int jq0 = 0, jq1 = 0;     // jobs issued per stream so far (phase of S_FULL / S_FREE)
        int s_owner = -1;         // stream whose scores were last written to S
        bool ok = true;
        auto wait = [&](int b, uint32_t par) -> bool { return mbar_wait_warp(bar(b), par, abort_flag, p.status); };
        static_assert(KST == 2, "two K stages are selected by a flag");
        const uint32_t qlo0 = desc_lo_kmajor(sQ), qlo1 = desc_lo_kmajor(sQ + TILE_BYTES);
        const uint32_t klo0 = desc_lo_kmajor(sK), klo1 = desc_lo_kmajor(sK + TILE_BYTES);
        for (int it = 0; it < n_my && ok; ++it) {
            const UnitInfo u = unit_of(it);
            if (u.ntiles == 0) continue;
            const bool two = u.two;
            const int njobs = two ? 2 * u.ntiles : u.ntiles;
            ok = wait(BAR_Q_FULL, au & 1);
            for (int k = 0; k < njobs && ok; ++k) {
                const int i = k & 1;
                const int r = kvc + (two ? (k >> 1) : k), st = r % KST;
                if (!two || i == 0) {
                    if (!(ok = wait(BAR_K_FULL + st, (r / KST) & 1))) break;
                }
                if (s_owner >= 0) {
                    // the previous job's scores must have left S
                    if (!(ok = wait(BAR_S_FREE + s_owner, (uint32_t)((s_owner ? jq1 : jq0) - 1) & 1u))) break;
                }
                tc_fence_after();
                tc_qk8(tmem + COL_S, (two && i) ? qlo1 : qlo0, st ? klo1 : klo0);
                tc_commit(bar(BAR_S_FULL + i));
                if (!two || i == 1) tc_commit(bar(BAR_K_EMPTY + st));
                if (k == njobs - 1) tc_commit(bar(BAR_Q_EMPTY));   // every QK^T of the unit is issued
                s_owner = i;
                if (i) ++jq1; else ++jq0;
            }
            kvc += u.ntiles;
            ++au;
        }
        // after an abort nothing this warp issued may still be running when TMEM is given back
        // (at a regular end the epilogues have waited for every MMA already)
        if (!ok) {
            tc_commit(bar(BAR_DRAIN + 0));
            mbar_wait_slow(bar(BAR_DRAIN + 0), 0, abort_flag, nullptr, true);
        }
    } else if (warp == 11) {
        // ------------------------------------------------------------ PV issuer (all lanes converged)
        // O_i += P_i V job by job: 8 k-steps of 16 keys, P (bf16 pairs) read from TMEM.  The
        // softmax hands P over in two halves of 64 keys, so the first four k-steps run while
        // the second half of the exponentials is still being computed.
        int kvc = 0;
        int au = 0, au1 = 0;      // non-empty units so far; those of them in which stream 1 had jobs
        int jp0 = 0, jp1 = 0;     // jobs issued per stream so far (phase of P_READY / P_FREE)
        bool ok = true;
        auto wait = [&](int b, uint32_t par) -> bool { return mbar_wait_warp(bar(b), par, abort_flag, p.status); };
        static_assert(VST == 2, "two V stages are selected by a flag");
        const uint32_t vlo0 = desc_lo_mnmajor(sV), vlo1 = desc_lo_mnmajor(sV + TILE_BYTES);
        for (int it = 0; it < n_my && ok; ++it) {
            const UnitInfo u = unit_of(it);
            if (u.ntiles == 0) continue;
            const bool two = u.two;
            const int njobs = two ? 2 * u.ntiles : u.ntiles;
            const int n1 = two ? u.ntiles : u.ntiles / 2;      // jobs of stream 1
            for (int k = 0; k < njobs && ok; ++k) {
                const int i = k & 1;
                const int r = kvc + (two ? (k >> 1) : k), st = r % VST;
                const bool first = k < 2;                      // first job of its stream in this unit
                const uint32_t par = (uint32_t)(i ? jp1 : jp0) & 1u;
                const uint32_t vlo = st ? vlo1 : vlo0;
                const uint32_t tP = tmem + (i ? COL_P1 : COL_P0), tO = tmem + (i ? COL_O1 : COL_O0);
                if (!two || i == 0) {
                    if (!(ok = wait(BAR_V_FULL + st, (r / VST) & 1))) break;
                }
                if (!(ok = wait(BAR_P_READY + i, par))) break;
                if (first && (i ? au1 : au) > 0) {
                    // the accumulator still belongs to the previous unit until its rows were read out
                    if (!(ok = wait(BAR_O_FREE + i, (uint32_t)((i ? au1 : au) - 1) & 1u))) break;
                }
                tc_fence_after();
                tc_pv4(tO, tP, vlo, first ? 0u : 1u);
                if (!(ok = wait(BAR_P_READY2 + i, par))) break;
                tc_fence_after();
                tc_pv4(tO, tP + 32, vlo + 4 * 128, 1u);
                tc_commit(bar(BAR_P_FREE + i));
                if (!two || i == 1) tc_commit(bar(BAR_V_EMPTY + st));
                if (k + 2 >= njobs) tc_commit(bar(BAR_O_DONE + i));   // the stream's last job of the unit
                if (i) ++jp1; else ++jp0;
            }
            kvc += u.ntiles;
            ++au;
            if (n1 > 0) ++au1;
        }
        if (!ok) {
            tc_commit(bar(BAR_DRAIN + 1));
            mbar_wait_slow(bar(BAR_DRAIN + 1), 0, abort_flag, nullptr, true);
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
        // ------------------------------------------------------------ softmax + epilogue
        const int i = warp >> 2;                         // stream of this warpgroup
        const int rloc = (warp & 3) * 32 + lane;         // row inside the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_addr + COL_S;
        const uint32_t tP = tmem + lane_addr + (i ? COL_P1 : COL_P0);
        const uint32_t tO = tmem + lane_addr + (i ? COL_O1 : COL_O0);
        int kvc = 0;      // key tiles of all non-empty units so far (ring position of the V tiles)
        int tcnt = 0;     // jobs this stream has processed so far (barrier phase)
        int auc = 0;      // non-empty units this stream has finished so far (barrier phase)
        int auc1 = 0;     // units in which stream 1 had jobs (phase of its barriers as seen by warpgroup 0)
        int mlc = 0;      // single-row-tile units whose odd-tile stream had tiles
        bool ok = true;
        for (int it = 0; it < n_my && ok; ++it) {
            const UnitInfo u = unit_of(it);
            const int ntiles = u.ntiles;
            // with one row tile only, the two warpgroups take the even / odd key tiles of the
            // same rows and warpgroup 0 merges the two partial results in the epilogue
            const bool alt = !u.two;
            const int my_n = alt ? (i == 0 ? (ntiles + 1) / 2 : ntiles / 2) : ntiles;
            const int n1 = alt ? ntiles / 2 : ntiles;           // tiles of stream 1 in this unit
            const int b = u.b, c = u.c;
            const int row = u.row0 + (alt ? 0 : i * BM) + rloc;
            const bool rvalid = row < R;
            if (warp == 0 && lane == 0) {
                const int Lraw = p.seq_lens[b];
                if ((Lraw < 0 || Lraw > p.Lmax) && p.status) atomicOr((unsigned*)p.status, GSD_DEV_BAD_SEQ_LEN);
            }
            float m_ref = -CUDART_INF_F, l_run = 0.f;
            const uint32_t* mrow = p.mask + ((size_t)b * N + (rvalid ? row / G : 0)) * p.W;
            for (int cnt = 0; cnt < my_n; ++cnt) {
                const int idx = alt ? 2 * cnt + i : cnt;
                const TileInfo ti = tile_info(u.t_begin + idx, u.nPT, u.L, u.live);
                // visibility words of this row for the 128 keys of the tile
                uint32_t mw[4];
                if (ti.kind == 0) {
                    mw[0] = mw[1] = mw[2] = mw[3] = 0xFFFFFFFFu;
                } else if (ti.kind == 1) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int from = (BN - ti.nvalid) - 32 * k;      // first visible key of the word
                        mw[k] = from <= 0 ? 0xFFFFFFFFu : (from >= 32 ? 0u : ~((1u << from) - 1u));
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int wi = (ti.key0 >> 5) + k;
                        uint32_t word = (rvalid && wi < p.W) ? mrow[wi] : 0u;
                        const int rem = N - 32 * wi;
                        if (rem < 32) word &= rem <= 0 ? 0u : ((1u << rem) - 1u);
                        mw[k] = word;
                    }
                }
                const uint32_t par = (uint32_t)((tcnt + cnt) & 1);
                ok = mbar_wait(bar(BAR_S_FULL + i), par, abort_flag, p.status);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();

                // the whole score row of this thread: 128 fp32 registers
                float sc[BN];
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) tc_ld32p(tS + ch * 32, sc + ch * 32);
                tc_wait_ld();
                tc_fence_before();
                if (lane == 0) mbar_arrive(bar(BAR_S_FREE + i));   // the next job's QK^T may overwrite S
                if (ti.kind != 0) {
#pragma unroll
                    for (int e = 0; e < BN; ++e) sc[e] = ((mw[e >> 5] >> (e & 31)) & 1u) ? sc[e] : -CUDART_INF_F;
                }
                float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
                for (int e = 0; e < BN; e += 8) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) mx4[k] = max3(mx4[k], sc[e + 2 * k], sc[e + 2 * k + 1]);
                }
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                const float m_tile = mx * p.scale_log2;     // scale > 0 keeps the order
                float m_new = m_ref, alpha = 1.f;
                bool need = false;
                if (m_ref == -CUDART_INF_F) {
                    m_new = m_tile;                         // nothing accumulated for this row yet
                } else if (m_tile > m_ref + kRescaleThreshold) {
                    m_new = m_tile;
                    alpha = fast_exp2(m_ref - m_new);
                    need = true;
                }
                if (__any_sync(0xFFFFFFFFu, need)) {
                    // once the PV of this stream's previous job has completed, the accumulator of
                    // this row is final for all earlier tiles: rescale it in place
                    ok = mbar_wait(bar(BAR_P_FREE + i), (uint32_t)((tcnt + cnt - 1) & 1), abort_flag, p.status);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int ch = 0; ch < 4; ++ch) {
                        float v[32];
                        tc_ld32(tO + ch * 32, v);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] *= alpha;
                        tc_st32(tO + ch * 32, v);
                    }
                    l_run *= alpha;
                }
                m_ref = m_new;
                const float m_use = m_ref == -CUDART_INF_F ? 0.f : m_ref;

                // P = 2^(s*scale - m) as bf16 pairs into the 64 columns of P_i; a masked score is
                // -inf and comes out as exactly 0
                const float2 scale2 = make_float2(p.scale_log2, p.scale_log2);
                const float2 negm2 = make_float2(-m_use, -m_use);
                float2 sum2[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};   // four chains
                uint32_t pk[4][16];
                auto exp_chunk = [&](int ch) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const float2 t = ffma2(make_float2(sc[ch * 32 + 2 * e], sc[ch * 32 + 2 * e + 1]), scale2, negm2);
                        const float2 pe = make_float2(fast_exp2(t.x), fast_exp2(t.y));
                        sum2[e & 3] = fadd2(sum2[e & 3], pe);
                        pk[ch][e] = pack_bf16(pe.x, pe.y);
                    }
                };
                // The TMEM stores of one half are in flight while the next chunk's exponentials are
                // computed; the hand-off of a half follows once its stores have landed.
                exp_chunk(0);
                exp_chunk(1);
                if (tcnt + cnt > 0) {
                    // P_i is still being read until the PV of this stream's previous job has completed
                    ok = mbar_wait(bar(BAR_P_FREE + i), (uint32_t)((tcnt + cnt - 1) & 1), abort_flag, p.status);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                }
                tc_st16(tP + 0, pk[0]);
                tc_st16(tP + 16, pk[1]);
                exp_chunk(2);
                tc_wait_st();              // keys 0..63 are in place (and any rescale of O is done)
                tc_fence_before();
                if (lane == 0) mbar_arrive(bar(BAR_P_READY + i));
                exp_chunk(3);
                tc_st16(tP + 32, pk[2]);
                tc_st16(tP + 48, pk[3]);
                l_run += ((sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y)) + ((sum2[2].x + sum2[2].y) + (sum2[3].x + sum2[3].y));
                tc_wait_st();
                tc_fence_before();
                if (lane == 0) mbar_arrive(bar(BAR_P_READY2 + i));
            }
            if (!ok) {
                // gave up inside the key loop: the warpgroup's decision barrier of this unit (below)
                // still has to see this warp, or the neighbours would wait there for ever
                if (u.nsplit == 1 && !(alt && i == 1)) wg_all(1 + i, false);
                break;
            }
            if (alt && i == 1) {
                // odd-tile stream: publish (max, sum); warpgroup 0 reads the accumulator itself
                if (my_n > 0) {
                    s_ml1[rloc] = make_float2(m_ref, l_run);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(BAR_ML_READY));
                    ++mlc;
                    ++auc;
                }
                kvc += ntiles;
                tcnt += my_n;
                continue;
            }
            // ---- epilogue: pull the accumulator row into registers, give TMEM back, then store
            // every wait of the epilogue first ...
            if (ntiles > 0) {
                ok = mbar_wait(bar(BAR_O_DONE + i), (uint32_t)(auc & 1), abort_flag, p.status);
                if (ok && alt && n1 > 0) {
                    ok = mbar_wait(bar(BAR_O_DONE + 1), (uint32_t)(auc1 & 1), abort_flag, p.status);
                    if (ok) ok = mbar_wait(bar(BAR_ML_READY), (uint32_t)(mlc & 1), abort_flag, p.status);
                }
                ok = __all_sync(0xFFFFFFFFu, ok);
            }
            if (u.nsplit == 1) {
                // ... then the four warps decide together whether to go on: the store section below
                // meets at hardware barriers, which have no time limit, so no warp may enter it while
                // a neighbour has given up.  Every warp of the warpgroup takes part in this barrier
                // once per unit, here or where it gave up.
                ok = wg_all(1 + i, ok);
            }
            if (!ok) break;
            float acc[HD];
            if (ntiles > 0) {
                tc_fence_after();
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) tc_ld32p(tO + ch * 32, acc + ch * 32);
                tc_wait_ld();
                if (alt && n1 > 0) {
                    // merge the odd-tile stream: O = w0 O0 + w1 O1, l = w0 l0 + w1 l1 at the common maximum
                    const float2 ml1 = s_ml1[rloc];
                    const float m = fmaxf(m_ref, ml1.x);
                    const float m_use = m == -CUDART_INF_F ? 0.f : m;
                    const float w0 = fast_exp2(m_ref - m_use), w1 = fast_exp2(ml1.x - m_use);
                    const uint32_t tO1 = tmem + lane_addr + COL_O1;
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        float v[32];
                        tc_ld32(tO1 + ch * 32, v);
                        tc_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) acc[ch * 32 + e] = w0 * acc[ch * 32 + e] + w1 * v[e];
                    }
                    l_run = w0 * l_run + w1 * ml1.y;
                    m_ref = m;
                    tc_fence_before();
                    if (lane == 0) mbar_arrive(bar(BAR_O_FREE + 1));
                    ++mlc;
                }
                tc_fence_before();
                if (lane == 0) mbar_arrive(bar(BAR_O_FREE + i));
            } else {
#pragma unroll
                for (int e = 0; e < HD; ++e) acc[e] = 0.f;
            }
            if (u.nsplit == 1) {
                // Normalise, round to bf16 and stage the rows in shared memory in the swizzled tile
                // layout; one thread then writes each 64-column half with a TMA tile store (full
                // 128-byte lines instead of 32 scattered 16-byte pieces per store instruction;
                // rows of nodes >= N are clipped by the tensor map).
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
                const uint32_t stage = sStage + (uint32_t)i * HALF_BYTES;
                unsigned char* srow = smem_raw + (stage - smem_u32(smem_raw)) + rloc * 128;
                const bool issuer = (warp & 3) == 0 && lane == 0;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int e = h * 64 + k * 8;
                        uint4 v;
                        v.x = pack_bf16(acc[e + 0] * inv, acc[e + 1] * inv);
                        v.y = pack_bf16(acc[e + 2] * inv, acc[e + 3] * inv);
                        v.z = pack_bf16(acc[e + 4] * inv, acc[e + 5] * inv);
                        v.w = pack_bf16(acc[e + 6] * inv, acc[e + 7] * inv);
                        *reinterpret_cast<uint4*>(srow + ((k ^ (rloc & 7)) << 4)) = v;
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    wg_barrier(1 + i);
                    if (issuer) {
                        tma_store_4d(&tm_out, stage, h * 64, c * G, (u.row0 + (alt ? 0 : i * BM)) / G, b);
                        bulk_commit();
                        bulk_wait_read();          // the staging block may be overwritten again
                    }
                    wg_barrier(1 + i);
                }
            } else if (rvalid) {
                {
                    const size_t prow = (size_t)u.slot * (2 * BM) + (alt ? 0 : i * BM) + rloc;
                    if (GSD_IN_BOUNDS(u.slot >= 0 && u.slot < p.slots, p.status)) {
                    float* dst = p.part_o + prow * HD;
#pragma unroll
                    for (int k = 0; k < HD / 4; ++k)
                        *reinterpret_cast<float4*>(dst + k * 4) =
                            make_float4(acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]);
                    *reinterpret_cast<float2*>(p.part_ml + prow * 2) = make_float2(m_ref, l_run);
                    }
                }
            }
            kvc += ntiles;
            tcnt += my_n;
            if (ntiles > 0) ++auc;
            if (n1 > 0) ++auc1;
        }
        if ((warp & 3) == 0 && lane == 0) bulk_wait_all();   // the output stores have landed
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 10) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !ptr) {
            if (e != cudaSuccess) set_cuda_error(e, "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)");
            else set_error_text("cuTensorMapEncodeTiled is not available in this driver");
            return nullptr;
        }
        fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

// [d3][d2][d1][D] bf16 tensor; box = 64 columns x box1 x box2 x 1, 128-byte swizzle, zero fill
int make_map(CUtensorMap* m, const void* base, uint64_t d1, uint64_t d2, uint64_t d3, uint32_t box1, uint32_t box2) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return GSD_ERR_CUDA;
    const cuuint64_t dims[4] = {(cuuint64_t)HD, d1, d2, d3};
    const cuuint64_t strides[3] = {(cuuint64_t)HD * 2, (cuuint64_t)HD * 2 * d1, (cuuint64_t)HD * 2 * d1 * d2};
    const cuuint32_t box[4] = {64, box1, box2, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        snprintf(msg, sizeof msg, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        set_error_text(msg);
        return GSD_ERR_CUDA;
    }
    return GSD_OK;
}

}  // namespace

bool attn_tcgen05_supports(int D, int G) { return D == HD && G >= 1 && G <= BM && BM % G == 0; }

int launch_attn_tcgen05(const AttnArgs& a) {
    if (!attn_tcgen05_supports(a.D, a.G)) {
        set_error_text("tcgen05 back end needs D == 128 and a group size that divides 128");
        return GSD_ERR_UNSUPPORTED;
    }
    CUtensorMap tq, tk, tv, tdk, tdv, tout;
    int rc;
    if ((rc = make_map(&tq, a.q, a.Hq, a.N, a.B, a.G, BM / a.G)) != GSD_OK) return rc;
    if ((rc = make_map(&tk, a.k_cache, a.Hkv, a.Lmax, a.B, 1, BN)) != GSD_OK) return rc;
    if ((rc = make_map(&tv, a.v_cache, a.Hkv, a.Lmax, a.B, 1, BN)) != GSD_OK) return rc;
    if ((rc = make_map(&tdk, a.draft_k, a.Hkv, a.N, a.B, 1, BN)) != GSD_OK) return rc;
    if ((rc = make_map(&tdv, a.draft_v, a.Hkv, a.N, a.B, 1, BN)) != GSD_OK) return rc;
    if ((rc = make_map(&tout, a.out, a.Hq, a.N, a.B, a.G, BM / a.G)) != GSD_OK) return rc;
    TcParams p;
    p.mask = a.mask; p.seq_lens = a.seq_lens; p.out = (__nv_bfloat16*)a.out; p.status = a.status;
    p.B = a.B; p.N = a.N; p.Hq = a.Hq; p.Hkv = a.Hkv; p.Lmax = a.Lmax; p.G = a.G; p.W = a.W;
    p.R = a.N * a.G; p.scale_log2 = a.scale_log2; p.plan = a.plan.dev;
    p.part_o = (float*)a.workspace;
    p.part_ml = (float*)((char*)a.workspace + plan_part_o_bytes(a.plan, a.D));
    {
        // the opt-in for large dynamic shared memory is per device and sticks: do it once
        static bool done[64] = {};
        int dev = 0;
        GSD_CUDA_TRY(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64 || !done[dev]) {
            GSD_CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
            if (dev >= 0 && dev < 64) done[dev] = true;
        }
    }
    p.total_work = a.plan.ctas;
    p.slots = a.plan.slots;
    p.wait_limit_ns = g_wait_limit_ns;
    p.withhold_first_k = g_withhold_first_k;
    DeviceInfo di;
    if (device_info(&di) != 0) return GSD_ERR_CUDA;
    p.bal_cta = nullptr;
    p.bal_units = nullptr;
    p.seq.hdr = nullptr; p.seq.nsplit = nullptr; p.seq.unit_off = nullptr; p.seq.slot_off = nullptr;
    if (a.plan.dev.balanced) {
        // one CTA per share of the table; the table is being written by the planning kernel,
        // beside which this kernel may start
        if (a.plan.dev.balanced == 2) {
            p.seq = plan_seq_table(a.plan, a.D, a.B, a.workspace);
        } else {
            const BalTable t = plan_bal_table(a.plan, a.D, a.workspace);
            p.bal_cta = t.cta;
            p.bal_units = t.units;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)a.plan.ctas);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = kSmemBytes;
        cfg.stream = a.stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        GSD_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_tc_kernel, tq, tk, tv, tdk, tdv, tout, p));
        return GSD_OK;
    }
    dim3 grid(a.plan.ctas < di.sm_count ? a.plan.ctas : di.sm_count);
    attn_tc_kernel<<<grid, kThreads, kSmemBytes, a.stream>>>(tq, tk, tv, tdk, tdv, tout, p);
    GSD_CUDA_TRY(cudaGetLastError());
    return GSD_OK;
}

void debug_attn_wait(unsigned long long limit_ns, int withhold_first_k) {
    g_wait_limit_ns = limit_ns ? limit_ns : kWaitLimitNs;
    g_withhold_first_k = withhold_first_k;
}

}  // namespace gsd
