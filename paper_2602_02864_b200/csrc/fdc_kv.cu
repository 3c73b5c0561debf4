// Slot-indexed KV append (Sec. 3.3: one shared cache, every emitted token's K/V written once
// at the row its fixed slot reserves; padding rows are never written).
#include "fdc_internal.h"

using namespace fdc;

#define FDC_CUDA(call)                                   \
    do {                                                 \
        cudaError_t e_ = (call);                         \
        if (e_ != cudaSuccess) return set_cuda_error(e_); \
    } while (0)

namespace {

// One block per branch slot, or a grid-stride loop over the slots when there are more slots than
// blocks; threads copy 16-byte vectors.
__global__ void __launch_bounds__(128) kv_append_kernel(char* __restrict__ k, char* __restrict__ v, int64_t stride_scene_b,
                                 int64_t stride_head_b, int64_t stride_row_b, int rows, int hkv, int row_bytes,
                                 int max_active, int n_slots, const int32_t* __restrict__ n_active,
                                 const int32_t* __restrict__ kv_row, const char* __restrict__ k_new,
                                 const char* __restrict__ v_new, int32_t* __restrict__ status)
{
    // Programmatic dependent launch.  The kernel after this one (the attention kernel) may be
    // scheduled as soon as every block of this grid is resident: its blocks then take the SMs as
    // they become free, set themselves up and wait for this grid to complete.  This grid waits for
    // the kernel before it, so completion still follows the stream order.  The grid is small (one
    // block of 128 threads or two of 64 per SM at most, 32 registers a thread) so that all of it can
    // be resident beside the attention blocks that are still running.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // All loads of a slot are issued before anything depends on them (the rows of idle branch
    // slots exist in k_new / v_new too, so they can be read before n_active is known): one trip
    // to memory instead of three in a row.
    const int vec_per_row = row_bytes >> 4, nvec = hkv * vec_per_row;
    for (int slot = blockIdx.x; slot < n_slots; slot += gridDim.x) {
        const int s = slot / max_active, b = slot - s * max_active;
        const size_t src0 = (size_t)slot * hkv * row_bytes;
        const int na = n_active[s];
        const int row = kv_row[slot];
        for (int i0 = threadIdx.x; i0 < nvec; i0 += 2 * blockDim.x) {
            const int i1 = i0 + blockDim.x;
            uint4 kk[2], vv[2];
            kk[0] = *reinterpret_cast<const uint4*>(k_new + src0 + (size_t)i0 * 16);
            vv[0] = *reinterpret_cast<const uint4*>(v_new + src0 + (size_t)i0 * 16);
            if (i1 < nvec) {
                kk[1] = *reinterpret_cast<const uint4*>(k_new + src0 + (size_t)i1 * 16);
                vv[1] = *reinterpret_cast<const uint4*>(v_new + src0 + (size_t)i1 * 16);
            }
            if (b >= na) break;
            if (row < 0 || row >= rows) {
                if (threadIdx.x == 0) atomicOr(status, FDC_DEV_ROW_RANGE);
                break;
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int i = j ? i1 : i0;
                if (i < nvec) {
                    const int g = i / vec_per_row, c = i - g * vec_per_row;
                    const size_t dst = (size_t)s * stride_scene_b + (size_t)g * stride_head_b + (size_t)row * stride_row_b + (size_t)c * 16;
                    *reinterpret_cast<uint4*>(k + dst) = kk[j];
                    *reinterpret_cast<uint4*>(v + dst) = vv[j];
                }
            }
        }
    }
}

// Pre-filled field-name rows (Sec. 3.1: every line starts "field name:"; Fig. 3: those tokens are
// "pre-filled"): fixed row i of a scene (fields in template order, then token order) goes to row
// P + base[v] + j of the cache.  One block per (scene, fixed row); threads copy 16-byte vectors.
__global__ void __launch_bounds__(128) kv_write_fixed_kernel(const PlanDev* __restrict__ plan, char* __restrict__ k, char* __restrict__ v,
                                                             int64_t stride_scene_b, int64_t stride_head_b, int64_t stride_row_b, int rows,
                                                             int hkv, int row_bytes, int n_fixed_total, const char* __restrict__ k_fixed,
                                                             const char* __restrict__ v_fixed, int32_t* __restrict__ status)
{
    const int s = blockIdx.x / n_fixed_total, i = blockIdx.x - s * n_fixed_total;
    __shared__ int s_row;
    if (threadIdx.x == 0) {
        int acc = 0, row = -1;
        for (int node = 0; node < plan->n; ++node) {
            const int nf = plan->nfixed[node];
            if (i < acc + nf) {
                row = plan->P + plan->base[node] + (i - acc);
                break;
            }
            acc += nf;
        }
        if (row < 0 || row >= rows) {
            atomicOr(status, FDC_DEV_ROW_RANGE);
            row = -1;
        }
        s_row = row;
    }
    __syncthreads();
    const int row = s_row;
    if (row < 0) return;
    const int vec_per_row = row_bytes >> 4, nvec = hkv * vec_per_row;
    for (int x = threadIdx.x; x < nvec; x += blockDim.x) {
        const int g = x / vec_per_row, c = x - g * vec_per_row;
        const size_t src = (((size_t)s * hkv + g) * n_fixed_total + i) * row_bytes + (size_t)c * 16;
        const size_t dst = (size_t)s * stride_scene_b + (size_t)g * stride_head_b + (size_t)row * stride_row_b + (size_t)c * 16;
        *reinterpret_cast<uint4*>(k + dst) = *reinterpret_cast<const uint4*>(k_fixed + src);
        *reinterpret_cast<uint4*>(v + dst) = *reinterpret_cast<const uint4*>(v_fixed + src);
    }
}

}  // namespace

namespace fdc {

int check_kv_desc(const fdc_plan* p, const fdc_kv_desc* kv, int32_t layer)
{
    if (!p || !kv) return FDC_ERR_NULL;
    if (!kv->k || !kv->v) return FDC_ERR_NULL;
    if (kv->dtype != FDC_F32 && kv->dtype != FDC_BF16) return FDC_ERR_DTYPE;
    if (kv->batch < 1 || kv->batch > FDC_MAX_BATCH || kv->layers < 1 || layer < 0 || layer >= kv->layers)
        return FDC_ERR_RANGE;
    if (kv->hkv < 1 || kv->hq < 1 || kv->hq % kv->hkv) return FDC_ERR_SHAPE;
    if (kv->head_dim != 64 && kv->head_dim != 128) return FDC_ERR_SHAPE;
    if (kv->rows < p->h.P + p->h.T) return FDC_ERR_SHAPE;
    if ((long long)p->h.max_active * (kv->hq / kv->hkv) > FDC_MAX_QROWS) return FDC_ERR_SHAPE;
    const int64_t st[4] = {kv->stride_scene, kv->stride_layer, kv->stride_head, kv->stride_row};
    for (int i = 0; i < 4; ++i)
        if (st[i] < 0 || (st[i] & 7)) return FDC_ERR_SHAPE;
    if (kv->stride_row < kv->head_dim) return FDC_ERR_SHAPE;
    if (((uintptr_t)kv->k & 15) || ((uintptr_t)kv->v & 15)) return FDC_ERR_SHAPE;
    return FDC_OK;
}

}  // namespace fdc

namespace fdc {

int launch_kv_append(fdc_plan* p, const fdc_kv_desc* kv, int32_t layer, const int32_t* d_n_active, const int32_t* d_kv_row,
                     const void* d_k_new, const void* d_v_new, void* stream)
{
    const int es = kv->dtype == FDC_F32 ? 4 : 2;
    char* kb = (char*)kv->k + (size_t)layer * kv->stride_layer * es;
    char* vb = (char*)kv->v + (size_t)layer * kv->stride_layer * es;
    const int row_bytes = kv->head_dim * es;
    int threads = kv->hkv * (row_bytes >> 4);
    const int n_slots = kv->batch * p->h.max_active;
    // blocks small enough to sit beside a resident attention block: one of 128 threads per SM, or two of 64
    const int per_sm = n_slots > p->sm_count ? 2 : 1;
    threads = threads > 128 / per_sm ? 128 / per_sm : ((threads + 31) & ~31);
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(n_slots < per_sm * p->sm_count ? n_slots : per_sm * p->sm_count);
        cfg.blockDim = dim3(threads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = (cudaStream_t)stream;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        FDC_CUDA(cudaLaunchKernelEx(&cfg, kv_append_kernel, kb, vb, (int64_t)(kv->stride_scene * es), (int64_t)(kv->stride_head * es),
                                    (int64_t)(kv->stride_row * es), (int)kv->rows, (int)kv->hkv, row_bytes, (int)p->h.max_active, n_slots, d_n_active,
                                    d_kv_row, (const char*)d_k_new, (const char*)d_v_new, p->d_status));
    }
    note_launch();
    return FDC_OK;
}

int flush_pending_append(fdc_plan* p)
{
    if (!p || !p->pend.valid) return FDC_OK;
    p->pend.valid = 0;
    return launch_kv_append(p, &p->pend.kv, p->pend.layer, p->pend.d_n_active, p->pend.d_kv_row, p->pend.d_k_new, p->pend.d_v_new,
                            p->pend.stream);
}

}  // namespace fdc

extern "C" int fdc_kv_append(fdc_plan* p, const fdc_kv_desc* kv, int32_t layer, const int32_t* d_n_active,
                             const int32_t* d_kv_row, const void* d_k_new, const void* d_v_new, void* stream)
{
    int rc = check_kv_desc(p, kv, layer);
    if (rc) return rc;
    if (!d_n_active || !d_kv_row || !d_k_new || !d_v_new) return FDC_ERR_NULL;
    if (((uintptr_t)d_k_new & 15) || ((uintptr_t)d_v_new & 15)) return FDC_ERR_SHAPE;
    rc = flush_pending_append(p);                 // an earlier recorded append never met its attention call
    if (rc) return rc;
    if (p->fuse_append && takes_tc_kernel(p, kv)) {
        // recorded only: the next fdc_decode_attn for this cache, layer and stream writes the rows itself
        fdc_pending_append& pe = const_cast<fdc_plan*>(p)->pend;
        pe.kv = *kv;
        pe.layer = layer;
        pe.d_n_active = d_n_active;
        pe.d_kv_row = d_kv_row;
        pe.d_k_new = d_k_new;
        pe.d_v_new = d_v_new;
        pe.stream = stream;
        pe.valid = 1;
        return FDC_OK;
    }
    return launch_kv_append(p, kv, layer, d_n_active, d_kv_row, d_k_new, d_v_new, stream);
}


extern "C" int fdc_kv_write_fixed(fdc_plan* p, const fdc_kv_desc* kv, int32_t layer, const void* d_k_fixed, const void* d_v_fixed,
                                  void* stream)
{
    int rc = check_kv_desc(p, kv, layer);
    if (rc) return rc;
    int total = 0;
    for (int v = 0; v < p->h.n; ++v) total += p->h.nfixed[v];
    if (total == 0) return FDC_OK;                 // the template has no pre-filled rows
    if (!d_k_fixed || !d_v_fixed) return FDC_ERR_NULL;
    if (((uintptr_t)d_k_fixed & 15) || ((uintptr_t)d_v_fixed & 15)) return FDC_ERR_SHAPE;
    rc = flush_pending_append(p);
    if (rc) return rc;
    const int es = kv->dtype == FDC_F32 ? 4 : 2;
    char* kb = (char*)kv->k + (size_t)layer * kv->stride_layer * es;
    char* vb = (char*)kv->v + (size_t)layer * kv->stride_layer * es;
    kv_write_fixed_kernel<<<kv->batch * total, 128, 0, (cudaStream_t)stream>>>(
        p->d, kb, vb, (int64_t)(kv->stride_scene * es), (int64_t)(kv->stride_head * es), (int64_t)(kv->stride_row * es), (int)kv->rows,
        (int)kv->hkv, kv->head_dim * es, total, (const char*)d_k_fixed, (const char*)d_v_fixed, p->d_status);
    note_launch();
    FDC_CUDA(cudaGetLastError());
    return FDC_OK;
}
