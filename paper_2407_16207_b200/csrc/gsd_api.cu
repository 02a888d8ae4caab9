// C ABI entry points of libgsd: argument validation, kernel selection, split planning,
// workspace layout, and the host-buffer step.  The arithmetic lives in the kernel files.
#include "gsd_internal.cuh"
#include <math.h>
#include <stdio.h>
#include <string.h>

namespace gsd {

static thread_local char g_err[256] = "";

void set_cuda_error(cudaError_t e, const char* where) {
    snprintf(g_err, sizeof g_err, "%s: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e), where);
    (void)cudaGetLastError();  // clear a non-sticky error so that the caller's next check is clean
}
void set_error_text(const char* text) { snprintf(g_err, sizeof g_err, "%s", text); }

int device_info(DeviceInfo* out) {
    static DeviceInfo cache[64];
    static bool have[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaGetDevice"); return -1; }
    if (dev >= 0 && dev < 64 && have[dev]) { *out = cache[dev]; return 0; }
    DeviceInfo di;
    e = cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&di.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) { set_cuda_error(e, "cudaDeviceGetAttribute"); return -1; }
    if (dev >= 0 && dev < 64) { cache[dev] = di; have[dev] = true; }
    *out = di;
    return 0;
}

static int attn_params_ok(const gsd_attn_params* p) {
    if (!p) return GSD_ERR_NULL_POINTER;
    if (p->B < 1 || p->N < 1 || p->N > GSD_MAX_NODES || p->Hq < 1 || p->Hkv < 1 ||
        p->Hq % p->Hkv != 0 || (p->D != 64 && p->D != 128) || p->Lmax < 1 || p->num_splits < GSD_ATTN_SPLIT_PER_SEQUENCE ||
        p->num_splits > 64)
        return GSD_ERR_BAD_SHAPE;
    if ((long long)p->B * p->Hkv > 65535) return GSD_ERR_BAD_SHAPE;
    if ((long long)p->N * (p->Hq / p->Hkv) > (1 << 20)) return GSD_ERR_BAD_SHAPE;
    if (p->kernel != GSD_ATTN_AUTO && p->kernel != GSD_ATTN_MMA && p->kernel != GSD_ATTN_TCGEN05)
        return GSD_ERR_BAD_SHAPE;
    if (p->kernel == GSD_ATTN_TCGEN05 && p->D != 128) return GSD_ERR_UNSUPPORTED;
    return GSD_OK;
}

int attn_pick_kernel(const gsd_attn_params* p) {
    if (p->kernel != GSD_ATTN_AUTO) return p->kernel;
    // the TMEM kernel pays off once the stacked rows fill its 128-row tiles
    const int G = p->Hq / p->Hkv;
    if (attn_tcgen05_supports(p->D, G) && p->N * G >= 64) return GSD_ATTN_TCGEN05;
    return GSD_ATTN_MMA;
}

AttnPlan attn_make_plan(const gsd_attn_params* p, int sm_count) {
    AttnPlan pl;
    pl.kernel = attn_pick_kernel(p);
    const bool tc = pl.kernel == GSD_ATTN_TCGEN05;
    const int G = p->Hq / p->Hkv;
    const int R = p->N * G;
    const int bn = tc ? 128 : 64;
    pl.rows_per_item = tc ? 256 : 64;
    pl.dev.tiles_per_unit = (R + pl.rows_per_item - 1) / pl.rows_per_item;
    pl.items = pl.dev.tiles_per_unit * p->B * p->Hkv;
    const int tiles = (p->Lmax + bn - 1) / bn + (p->N + bn - 1) / bn;
    int max_split = tiles / 4;                     // keep at least four key tiles per split
    if (max_split > 32) max_split = 32;
    if (max_split < 1) max_split = 1;
    const int resident = sm_count * (tc ? 1 : 3);  // CTAs the device holds at once
    pl.dev.items_a = pl.items;
    pl.dev.splits_a = 1;
    pl.dev.splits_b = 1;
    pl.dev.balanced = 0;
    // Shares of key tiles dealt out on the device from the true sequence lengths: on request
    // only.  Every cut costs a partial result (an fp32 accumulator tile written and read back,
    // as much traffic as a key tile), so it pays when the lengths of a batch differ by far
    // more than a share - one long context among short ones - and loses otherwise.
    const int tpu = pl.dev.tiles_per_unit;
    if (tc && p->num_splits == GSD_ATTN_SPLIT_BALANCED && resident <= 1024 && tpu <= resident &&
        (long long)pl.items * tiles < (1ll << 30)) {
        pl.dev.balanced = 1;
        // one group of tpu CTAs (a CTA per row-tile item) per share of the line
        const long long line = (long long)(pl.items / tpu) * tiles;   // tiles at full length
        const int groups = (int)(line < resident / tpu ? line : resident / tpu);
        pl.ctas = groups * tpu;
        pl.slots = 2 * pl.ctas;                                        // a CTA's first and last unit
        pl.ws_bytes = plan_part_o_bytes(pl, p->D) + plan_part_ml_bytes(pl) + plan_bal_bytes(pl, p->B);
        return pl;
    }
    if (tc && p->num_splits == GSD_ATTN_SPLIT_PER_SEQUENCE && resident <= 1024) {
        // split counts per sequence, chosen on the device; persistent CTAs walk the units
        pl.dev.balanced = 2;
        pl.ctas = resident;
        // slots: a sequence is cut when its tiles / target rounds to two or more, i.e. is at least
        // 1.5, and then gets at most tiles / target + 0.5 <= 4/3 tiles / target ranges per item;
        // tiles / target summed over everything is at most the units aimed at
        const long long bound = (4ll * kSeqPlanWaves * resident + 2) / 3 + 1;
        const long long cap = (long long)pl.items * kSeqPlanMaxSplit;
        pl.slots = (int)(bound < cap ? bound : cap);
        pl.ws_bytes = plan_part_o_bytes(pl, p->D) + plan_part_ml_bytes(pl) + plan_bal_bytes(pl, p->B);
        return pl;
    }
    if (p->num_splits > 0) {
        pl.dev.splits_a = p->num_splits;
    } else if (pl.items < resident) {
        int s = resident / pl.items;
        pl.dev.splits_a = s < max_split ? s : max_split;
    } else if (tc) {
        // whole items fill complete waves; the items of the last, partial wave are cut so that
        // they cover the machine once more instead of leaving most of it idle
        const int r = pl.items % resident;
        if (r > 0) {
            int s = resident / r;
            if (s > max_split) s = max_split;
            if (s > 1) {
                pl.dev.items_a = pl.items - r;
                pl.dev.splits_b = s;
            }
        }
    }
    const int items_b = pl.items - pl.dev.items_a;
    pl.ctas = pl.dev.items_a * pl.dev.splits_a + items_b * pl.dev.splits_b;
    pl.slots = (pl.dev.splits_a > 1 ? pl.dev.items_a * pl.dev.splits_a : 0) +
               (pl.dev.splits_b > 1 ? items_b * pl.dev.splits_b : 0);
    pl.ws_bytes = pl.slots ? plan_part_o_bytes(pl, p->D) + plan_part_ml_bytes(pl) : 0;
    return pl;
}

}  // namespace gsd

using namespace gsd;

extern "C" int gsd_version(void) { return GSD_VERSION; }

extern "C" void gsd_debug_attn_wait(uint64_t limit_ns, int32_t withhold_first_k) {
    debug_attn_wait((unsigned long long)limit_ns, (int)withhold_first_k);
}

extern "C" const char* gsd_status_string(int s) {
    switch (s) {
        case GSD_OK: return "ok";
        case GSD_ERR_NULL_POINTER: return "a required pointer is NULL";
        case GSD_ERR_BAD_SHAPE: return "unsupported or inconsistent sizes";
        case GSD_ERR_MISALIGNED: return "a tensor base is misaligned";
        case GSD_ERR_WORKSPACE: return "workspace missing or too small";
        case GSD_ERR_CUDA: return "a CUDA call failed";
        case GSD_ERR_UNSUPPORTED: return "the requested kernel cannot run this shape";
        default: return "unknown status";
    }
}

extern "C" const char* gsd_last_cuda_error(void) { return g_err; }

extern "C" int gsd_verify_attn_num_splits(const gsd_attn_params* p) {
    if (attn_params_ok(p) != GSD_OK) return 0;
    DeviceInfo di;
    if (device_info(&di) != 0) return 0;
    const AttnPlan pl = attn_make_plan(p, di.sm_count);
    if (pl.dev.balanced) return pl.dev.balanced == 2 ? GSD_ATTN_SPLIT_PER_SEQUENCE : GSD_ATTN_SPLIT_BALANCED;
    return pl.dev.splits_a > pl.dev.splits_b ? pl.dev.splits_a : pl.dev.splits_b;
}

extern "C" size_t gsd_verify_attn_workspace_bytes(const gsd_attn_params* p) {
    if (attn_params_ok(p) != GSD_OK) return 0;
    DeviceInfo di;
    if (device_info(&di) != 0) return 0;
    return attn_make_plan(p, di.sm_count).ws_bytes;
}

extern "C" int gsd_verify_attn(const void* q, const void* k_cache, const void* v_cache,
                               const void* draft_k, const void* draft_v,
                               const uint32_t* ancestor_mask, const int32_t* seq_lens, void* out,
                               const gsd_attn_params* p, void* workspace, size_t workspace_bytes,
                               int32_t* status, void* stream) {
    if (!p || !q || !k_cache || !v_cache || !draft_k || !draft_v || !ancestor_mask || !seq_lens || !out)
        return GSD_ERR_NULL_POINTER;
    const int ok = attn_params_ok(p);
    if (ok != GSD_OK) return ok;
    const void* ptrs[] = {q, k_cache, v_cache, draft_k, draft_v, out};
    for (const void* ptr : ptrs)
        if (((uintptr_t)ptr & 15u) != 0) return GSD_ERR_MISALIGNED;
    if (((uintptr_t)ancestor_mask & 3u) != 0 || ((uintptr_t)seq_lens & 3u) != 0) return GSD_ERR_MISALIGNED;
    DeviceInfo di;
    if (device_info(&di) != 0) return GSD_ERR_CUDA;
    const AttnPlan plan = attn_make_plan(p, di.sm_count);
    const size_t need = plan.ws_bytes;
    if (need > 0) {
        if (!workspace || workspace_bytes < need) return GSD_ERR_WORKSPACE;
        if (((uintptr_t)workspace & 255u) != 0) return GSD_ERR_MISALIGNED;
    }
    AttnArgs a;
    a.q = q; a.k_cache = k_cache; a.v_cache = v_cache; a.draft_k = draft_k; a.draft_v = draft_v;
    a.mask = ancestor_mask; a.seq_lens = seq_lens; a.out = out;
    a.B = p->B; a.N = p->N; a.Hq = p->Hq; a.Hkv = p->Hkv; a.D = p->D; a.Lmax = p->Lmax;
    a.G = p->Hq / p->Hkv; a.W = (p->N + 31) / 32;
    const float scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->D);
    a.scale_log2 = scale * 1.4426950408889634f;
    a.plan = plan; a.workspace = workspace; a.status = status;
    a.stream = (cudaStream_t)stream;
    int rc = GSD_OK;
    if (plan.dev.balanced && (rc = launch_attn_plan(a)) != GSD_OK) return rc;
    rc = plan.kernel == GSD_ATTN_TCGEN05 ? launch_attn_tcgen05(a) : launch_attn_mma(a);
    if (rc != GSD_OK) return rc;
    if (plan.slots > 0) rc = launch_attn_merge(a);
    return rc;
}

// ---------------------------------------------------------------- host-buffer step
namespace {
struct ArenaLayout {
    size_t q, kc, vc, dk, dv, mask, sl, out, logits, tok, pptr, pidx, atok, alen, anodes, status,
        ws_attn, ws_acc, total;
    size_t b_q, b_kv, b_d, b_mask, b_sl, b_logits, b_tok, b_pptr, b_pidx, b_acc, b_len;
};

bool arena_layout(const gsd_attn_params* ap, const gsd_accept_params* cp, ArenaLayout* L) {
    if (!ap || !cp || ap->B != cp->B || ap->N != cp->N) return false;
    const size_t B = ap->B, N = ap->N;
    L->b_q = B * N * ap->Hq * ap->D * 2;
    L->b_kv = B * (size_t)ap->Lmax * ap->Hkv * ap->D * 2;
    L->b_d = B * N * ap->Hkv * ap->D * 2;
    L->b_mask = B * N * ((N + 31) / 32) * 4;
    L->b_sl = B * 4;
    L->b_logits = B * N * (size_t)cp->V * 4;
    L->b_tok = B * N * 4;
    L->b_pptr = B * (N + 1) * 4;
    L->b_pidx = B * (size_t)cp->Ecap * 4;
    L->b_acc = B * (size_t)cp->Tcap * 4;
    L->b_len = B * 4;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L->q = take(L->b_q); L->kc = take(L->b_kv); L->vc = take(L->b_kv); L->dk = take(L->b_d);
    L->dv = take(L->b_d); L->mask = take(L->b_mask); L->sl = take(L->b_sl); L->out = take(L->b_q);
    L->logits = take(L->b_logits); L->tok = take(L->b_tok); L->pptr = take(L->b_pptr);
    L->pidx = take(L->b_pidx); L->atok = take(L->b_acc); L->alen = take(L->b_len);
    L->anodes = take(L->b_acc); L->status = take(4);
    L->ws_attn = take(gsd_verify_attn_workspace_bytes(ap));
    L->ws_acc = take(gsd_accept_workspace_bytes(cp));
    L->total = off;
    return true;
}
}  // namespace

extern "C" size_t gsd_verify_step_host_arena_bytes(const gsd_attn_params* ap, const gsd_accept_params* cp) {
    ArenaLayout L;
    if (attn_params_ok(ap) != GSD_OK || !cp || cp->V < 1 || cp->Ecap < 1 || cp->Tcap < 1) return 0;
    if (!arena_layout(ap, cp, &L)) return 0;
    return L.total;
}

namespace {
// One copy stream and three events per device, created at the first host-step call on that
// device and kept for the life of the process.
struct HostStepStreams {
    cudaStream_t copy = nullptr;
    cudaEvent_t entered = nullptr, attn_in = nullptr, accept_in = nullptr;
};
HostStepStreams* host_step_streams() {
    static HostStepStreams per_dev[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        gsd::set_error_text("gsd_verify_step_host: no current device");
        return nullptr;
    }
    HostStepStreams* h = &per_dev[dev];
    if (!h->copy) {
        cudaStream_t s = nullptr;
        cudaEvent_t e[3] = {nullptr, nullptr, nullptr};
        cudaError_t err = cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking);
        for (int i = 0; i < 3 && err == cudaSuccess; ++i) err = cudaEventCreateWithFlags(&e[i], cudaEventDisableTiming);
        if (err != cudaSuccess) {
            gsd::set_cuda_error(err, "gsd_verify_step_host: copy stream / events");
            return nullptr;
        }
        h->entered = e[0]; h->attn_in = e[1]; h->accept_in = e[2];
        h->copy = s;
    }
    return h;
}
}  // namespace

extern "C" int gsd_verify_step_host(const void* q, const void* k_cache, const void* v_cache,
                                    const void* draft_k, const void* draft_v,
                                    const uint32_t* ancestor_mask, const int32_t* seq_lens, void* out,
                                    const gsd_attn_params* ap, const float* logits,
                                    const int32_t* draft_tokens, const int32_t* parent_ptr,
                                    const int32_t* parent_idx, int32_t* accepted_tokens,
                                    int32_t* accepted_len, int32_t* accepted_nodes,
                                    const gsd_accept_params* cp, void* arena, size_t arena_bytes,
                                    int32_t* device_status_out, void* stream) {
    if (!ap || !cp || !q || !k_cache || !v_cache || !draft_k || !draft_v || !ancestor_mask ||
        !seq_lens || !out || !logits || !draft_tokens || !parent_ptr || !parent_idx ||
        !accepted_tokens || !accepted_len || !arena)
        return GSD_ERR_NULL_POINTER;
    const int ok = attn_params_ok(ap);
    if (ok != GSD_OK) return ok;
    // everything gsd_accept would refuse is refused here, before a byte is copied
    if (cp->B < 1 || cp->N < 1 || cp->N > GSD_MAX_NODES || cp->V < 1 || cp->Ecap < 1 || cp->Tcap < 1)
        return GSD_ERR_BAD_SHAPE;
    ArenaLayout L;
    if (!arena_layout(ap, cp, &L)) return GSD_ERR_BAD_SHAPE;
    if (arena_bytes < L.total) return GSD_ERR_WORKSPACE;
    if (((uintptr_t)arena & 255u) != 0) return GSD_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)arena;
    // The host->device copies go out on a copy stream of the library's own, the attention inputs
    // first; `stream` runs the attention as soon as those have landed and sends its output back
    // (the other direction of the link) while the logits are still coming in.
    HostStepStreams* hs = host_step_streams();
    if (!hs) return GSD_ERR_CUDA;
    cudaStream_t cs = hs->copy;
    int32_t dev_status = 0;
    // From here on work is in flight on both streams: whatever goes wrong, both are drained before
    // the call returns, so that the caller's host buffers and the arena are free again.
    auto enqueue = [&]() -> int {
    GSD_CUDA_TRY(cudaEventRecord(hs->entered, st));           // the arena may still be in use by earlier work on `stream`
    GSD_CUDA_TRY(cudaStreamWaitEvent(cs, hs->entered, 0));
    auto h2d = [&](size_t off, const void* src, size_t bytes) {
        return cudaMemcpyAsync(base + off, src, bytes, cudaMemcpyHostToDevice, cs);
    };
    GSD_CUDA_TRY(h2d(L.q, q, L.b_q));
    GSD_CUDA_TRY(h2d(L.kc, k_cache, L.b_kv));
    GSD_CUDA_TRY(h2d(L.vc, v_cache, L.b_kv));
    GSD_CUDA_TRY(h2d(L.dk, draft_k, L.b_d));
    GSD_CUDA_TRY(h2d(L.dv, draft_v, L.b_d));
    GSD_CUDA_TRY(h2d(L.mask, ancestor_mask, L.b_mask));
    GSD_CUDA_TRY(h2d(L.sl, seq_lens, L.b_sl));
    GSD_CUDA_TRY(cudaEventRecord(hs->attn_in, cs));
    GSD_CUDA_TRY(h2d(L.logits, logits, L.b_logits));
    GSD_CUDA_TRY(h2d(L.tok, draft_tokens, L.b_tok));
    GSD_CUDA_TRY(h2d(L.pptr, parent_ptr, L.b_pptr));
    GSD_CUDA_TRY(h2d(L.pidx, parent_idx, L.b_pidx));
    GSD_CUDA_TRY(cudaEventRecord(hs->accept_in, cs));
    GSD_CUDA_TRY(cudaMemsetAsync(base + L.status, 0, 4, st));
    GSD_CUDA_TRY(cudaStreamWaitEvent(st, hs->attn_in, 0));
    int rc = gsd_verify_attn(base + L.q, base + L.kc, base + L.vc, base + L.dk, base + L.dv,
                             (const uint32_t*)(base + L.mask), (const int32_t*)(base + L.sl),
                             base + L.out, ap, base + L.ws_attn,
                             gsd_verify_attn_workspace_bytes(ap), (int32_t*)(base + L.status), stream);
    if (rc != GSD_OK) return rc;
    GSD_CUDA_TRY(cudaMemcpyAsync(out, base + L.out, L.b_q, cudaMemcpyDeviceToHost, st));
    GSD_CUDA_TRY(cudaStreamWaitEvent(st, hs->accept_in, 0));
    rc = gsd_accept((const float*)(base + L.logits), (const int32_t*)(base + L.tok),
                    (const int32_t*)(base + L.pptr), (const int32_t*)(base + L.pidx),
                    (int32_t*)(base + L.atok), (int32_t*)(base + L.alen),
                    (int32_t*)(base + L.anodes), cp, base + L.ws_acc,
                    gsd_accept_workspace_bytes(cp), (int32_t*)(base + L.status), stream);
    if (rc != GSD_OK) return rc;
    GSD_CUDA_TRY(cudaMemcpyAsync(accepted_tokens, base + L.atok, L.b_acc, cudaMemcpyDeviceToHost, st));
    GSD_CUDA_TRY(cudaMemcpyAsync(accepted_len, base + L.alen, L.b_len, cudaMemcpyDeviceToHost, st));
    if (accepted_nodes)
        GSD_CUDA_TRY(cudaMemcpyAsync(accepted_nodes, base + L.anodes, L.b_acc, cudaMemcpyDeviceToHost, st));
    GSD_CUDA_TRY(cudaMemcpyAsync(&dev_status, base + L.status, 4, cudaMemcpyDeviceToHost, st));
    return GSD_OK;
    };
    const int rc_enqueue = enqueue();
    const cudaError_t e_copy = cudaStreamSynchronize(cs), e_main = cudaStreamSynchronize(st);
    if (rc_enqueue != GSD_OK) return rc_enqueue;
    if (e_copy != cudaSuccess) { set_cuda_error(e_copy, "cudaStreamSynchronize(copy stream)"); return GSD_ERR_CUDA; }
    if (e_main != cudaSuccess) { set_cuda_error(e_main, "cudaStreamSynchronize(stream)"); return GSD_ERR_CUDA; }
    if (device_status_out) *device_status_out = dev_status;
    return GSD_OK;
}
