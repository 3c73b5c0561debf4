// fdc_decode_attn: argument checks, kernel selection, split pass + combine pass.
#include <cmath>
#include <vector>

#include "fdc_internal.h"

using namespace fdc;

namespace {

// Upper bound of split CTAs any kernel variant uses (2 per SM), so that the workspace size
// does not depend on the variant.
inline int max_ctas(const fdc_plan* p) { return 2 * p->sm_count; }

inline size_t ws_bytes_for(const fdc_plan* p, const fdc_kv_desc* kv)
{
    const size_t slots = (size_t)max_ctas(p) + (size_t)kv->batch * kv->hkv;
    const size_t mmax = (size_t)p->h.max_active * (kv->hq / kv->hkv);
    size_t b = slots * mmax * (kv->head_dim + 2) * sizeof(float);
    return (b + 255) & ~(size_t)255;
}

struct Prof {
    std::vector<cudaEvent_t> ev;      // 3 per recorded call
    size_t used = 0;                  // events handed out since the last read
    static constexpr size_t kMaxCalls = 16384;
    cudaEvent_t next()
    {
        if (used == ev.size()) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
            ev.push_back(e);
        }
        return ev[used++];
    }
};

}  // namespace

namespace fdc {
void prof_destroy(fdc_plan* p)
{
    Prof* pr = (Prof*)p->prof;
    if (!pr) return;
    for (cudaEvent_t e : pr->ev) cudaEventDestroy(e);
    delete pr;
    p->prof = nullptr;
}

// The conditions under which fdc_decode_attn runs the tcgen05 kernel with the combine fused in
// (the only kernel that can also carry out a recorded append).
bool takes_tc_kernel(const fdc_plan* p, const fdc_kv_desc* kv)
{
    return kv->dtype == FDC_BF16 && kv->head_dim == 128 && (p->attn_kernel == 0 || p->attn_kernel == 3) &&
           (long long)p->h.max_active * (kv->hq / kv->hkv) <= 128 && (long long)kv->batch * kv->hkv <= FDC_PAIR_COUNTERS;
}
}  // namespace fdc

extern "C" {

int fdc_profile(fdc_plan* p, int32_t enable)
{
    if (!p) return FDC_ERR_NULL;
    if (enable && !p->prof) p->prof = new Prof;
    p->prof_on = enable != 0;
    return FDC_OK;
}

int fdc_profile_read(fdc_plan* p, float* split_ms, float* combine_ms, int32_t* calls)
{
    if (!p || !split_ms || !combine_ms || !calls) return FDC_ERR_NULL;
    *split_ms = *combine_ms = 0.f;
    *calls = 0;
    Prof* pr = (Prof*)p->prof;
    if (!pr) return FDC_OK;
    for (size_t i = 0; i + 2 < pr->used; i += 3) {
        cudaError_t e = cudaEventSynchronize(pr->ev[i + 2]);
        float a = 0.f, b = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&a, pr->ev[i], pr->ev[i + 1]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&b, pr->ev[i + 1], pr->ev[i + 2]);
        if (e != cudaSuccess) return set_cuda_error(e);
        *split_ms += a;
        *combine_ms += b;
        *calls += 1;
    }
    pr->used = 0;
    return FDC_OK;
}

int fdc_attn_workspace_bytes(const fdc_plan* p, const fdc_kv_desc* kv, size_t* bytes)
{
    if (!bytes) return FDC_ERR_NULL;
    int rc = check_kv_desc(p, kv, 0);
    if (rc) return rc;
    *bytes = ws_bytes_for(p, kv);
    return FDC_OK;
}

int fdc_set_fused_append(fdc_plan* p, int32_t on)
{
    if (!p) return FDC_ERR_NULL;
    int rc = flush_pending_append(p);
    if (rc) return rc;
    p->fuse_append = on ? 1 : 0;
    return FDC_OK;
}

int fdc_set_attn_kernel(fdc_plan* p, int32_t which)
{
    if (p) {
        int rcf = flush_pending_append(p);
        if (rcf) return rcf;
    }
    if (!p) return FDC_ERR_NULL;
    if (which < 0 || which > 3) return FDC_ERR_RANGE;
    p->attn_kernel = which;
    return FDC_OK;
}

const char* fdc_kernel_name(int32_t which)
{
    switch (which) {
        case 0: return "auto";
        case 1: return "ref_cuda_core";
        case 2: return "tma_mma_bf16";
        case 3: return "tma_tcgen05_bf16";
        default: return nullptr;
    }
}

int fdc_decode_attn(fdc_plan* p, const fdc_kv_desc* kv, int32_t layer, const int32_t* d_n_active,
                    const uint64_t* d_mask, const int32_t* d_tiles, const int32_t* d_ntiles, const void* d_q,
                    void* d_out, float scale, void* d_workspace, size_t ws_bytes, void* stream)
{
    int rc = check_kv_desc(p, kv, layer);
    if (rc) return rc;
    if (!d_n_active || !d_mask || !d_tiles || !d_ntiles || !d_q || !d_out) return FDC_ERR_NULL;
    if (!d_workspace || ((uintptr_t)d_workspace & 255) || ws_bytes < ws_bytes_for(p, kv)) return FDC_ERR_WORKSPACE;
    if (((uintptr_t)d_q & 15) || ((uintptr_t)d_out & 15)) return FDC_ERR_SHAPE;
    if (!(scale > 0.f) || !std::isfinite(scale)) return FDC_ERR_RANGE;
    const int es = kv->dtype == FDC_F32 ? 4 : 2;
    // a recorded append is carried out by this call's kernel if it belongs to it, else on its own first
    fdc_pending_append app = p->pend;
    if (app.valid) {
        const bool mine = takes_tc_kernel(p, kv) && app.kv.k == kv->k && app.kv.v == kv->v && app.layer == layer &&
                          app.stream == stream && app.d_n_active == d_n_active && app.kv.stride_layer == kv->stride_layer;
        if (mine) {
            p->pend.valid = 0;
        } else {
            rc = flush_pending_append(p);
            if (rc) return rc;
            app.valid = 0;
        }
    }

    AttnParams a;
    a.k = (const char*)kv->k + (size_t)layer * kv->stride_layer * es;
    a.v = (const char*)kv->v + (size_t)layer * kv->stride_layer * es;
    a.stride_scene = kv->stride_scene;
    a.stride_head = kv->stride_head;
    a.stride_row = kv->stride_row;
    a.q = d_q;
    a.out = d_out;
    a.mask = d_mask;
    a.tiles = d_tiles;
    a.ntiles = d_ntiles;
    a.n_active = d_n_active;
    a.batch = kv->batch;
    a.hkv = kv->hkv;
    a.hq = kv->hq;
    a.group = kv->hq / kv->hkv;
    a.max_active = p->h.max_active;
    a.mmax = a.max_active * a.group;
    a.W = p->h.W;
    a.P = p->h.P;
    a.rows = kv->rows;
    a.ntile_max = p->h.ntile_max;
    a.scale_log2 = scale * 1.4426950408889634f;
    const size_t slots = (size_t)max_ctas(p) + (size_t)kv->batch * kv->hkv;
    a.ws_o = (float*)d_workspace;
    a.ws_ml = a.ws_o + slots * a.mmax * kv->head_dim;
    a.n_cta = p->sm_count;
    a.status = p->d_status;
    a.app_row = nullptr;
    a.app_k = a.app_v = nullptr;

    cudaStream_t st = (cudaStream_t)stream;
    Prof* pr = p->prof_on ? (Prof*)p->prof : nullptr;
    if (pr && pr->used + 3 > 3 * Prof::kMaxCalls) pr = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr, e2 = nullptr;
    if (pr) {
        e0 = pr->next();
        e1 = pr->next();
        e2 = pr->next();
        if (!e0 || !e1 || !e2) return set_cuda_error(cudaErrorMemoryAllocation);
        cudaEventRecord(e0, st);
    }
    rc = FDC_ERR_SHAPE;
    a.pair_cnt = nullptr;
    a.split_memo = nullptr;
    a.seq = 0;
    a.early = 0;
    bool fused = false;                 // the split kernel merged the partials itself
    if (kv->dtype == FDC_BF16 && (p->attn_kernel == 0 || p->attn_kernel == 3)) {
        if ((long long)kv->batch * kv->hkv <= FDC_PAIR_COUNTERS) a.pair_cnt = p->d_pair_cnt;
        a.split_memo = (a.pair_cnt && kv->batch <= FDC_MEMO_BATCH && a.n_cta <= FDC_MEMO_CTAS) ? p->d_split_memo : nullptr;
        // The work split depends only on the pass tables, so it is computed once per pass, by a launch
        // of its own ahead of the pass's first attention launch (an ordinary launch: it begins after
        // everything before it in the stream has completed).
        bool split_now = false;
        if (a.split_memo) {
            const fdc_split_key& k = p->split_key;
            split_now = !k.valid || k.tables_gen != p->tables_gen || k.d_n_active != d_n_active || k.d_ntiles != d_ntiles ||
                        k.batch != kv->batch || k.hkv != kv->hkv || k.n_cta != a.n_cta || k.P != a.P || k.stream != stream;
            if (split_now) {
                a.seq = ++p->split_gen;
                a.early = 0;
                rc = launch_attn_tc_split(a, kv->head_dim, st);
                if (rc == FDC_OK) {
                    p->split_key = fdc_split_key{p->tables_gen, d_n_active, d_ntiles, kv->batch, kv->hkv, a.n_cta, a.P, stream, 1};
                } else {
                    p->split_key.valid = 0;
                    a.split_memo = nullptr;
                    split_now = false;
                }
                rc = FDC_ERR_SHAPE;
            }
            a.seq = p->split_gen;
        }
        // Reading ahead of the dependency wait: allowed from the second attention launch of a pass on
        // the same stream.  The first one waits for everything before it (the pass tables, the split)
        // before it lets the next kernel begin, and no kernel begins before the one ahead of it in the
        // stream has let it, so whatever runs later finds those complete.
        a.early = (!split_now && p->attn_gen == p->tables_gen && p->attn_stream == stream && p->attn_gen_valid) ? 1 : 0;
        if (app.valid) {
            a.app_row = app.d_kv_row;
            a.app_k = app.d_k_new;
            a.app_v = app.d_v_new;
        }
        rc = launch_attn_tc(a, kv->head_dim, st);
        if (rc == FDC_OK) {
            p->attn_gen = p->tables_gen;
            p->attn_stream = stream;
            p->attn_gen_valid = 1;
        }
        a.app_row = nullptr;
        if (app.valid && rc != FDC_OK) {
            // the kernel that would have written the rows was not launched: append on its own after all
            int rca = launch_kv_append(p, kv, layer, app.d_n_active, app.d_kv_row, app.d_k_new, app.d_v_new, stream);
            if (rca) return rca;
        }
        fused = rc == FDC_OK && a.pair_cnt != nullptr;
        a.pair_cnt = nullptr;
        a.split_memo = nullptr;
    }
    if (kv->dtype == FDC_BF16 && (p->attn_kernel == 2 || (rc == FDC_ERR_SHAPE && p->attn_kernel != 1)))
        rc = launch_attn_mma(a, kv->head_dim, st);
    if (rc == FDC_ERR_SHAPE) rc = launch_attn_ref(a, kv->dtype, kv->head_dim, st);
    if (rc) return rc;
    if (pr) cudaEventRecord(e1, st);
    if (!fused) rc = launch_attn_combine(a, kv->dtype, kv->head_dim, st);
    if (pr) cudaEventRecord(e2, st);
    return rc;
}

}  // extern "C"
