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

// grid.x = batch * max_active (one block per branch slot); threads copy 16-byte vectors.
__global__ void kv_append_kernel(char* __restrict__ k, char* __restrict__ v, int64_t stride_scene_b,
                                 int64_t stride_head_b, int64_t stride_row_b, int rows, int hkv, int row_bytes,
                                 int max_active, const int32_t* __restrict__ n_active,
                                 const int32_t* __restrict__ kv_row, const char* __restrict__ k_new,
                                 const char* __restrict__ v_new, int32_t* __restrict__ status)
{
    // programmatic dependent launch (see the attention kernel): wait for the kernel before this one,
    // let the one after it be scheduled
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int s = blockIdx.x / max_active, b = blockIdx.x - s * max_active;
    if (b >= n_active[s]) return;
    const int row = kv_row[blockIdx.x];
    if (row < 0 || row >= rows) {
        if (threadIdx.x == 0) atomicOr(status, FDC_DEV_ROW_RANGE);
        return;
    }
    const int vec_per_row = row_bytes >> 4;
    const size_t src0 = (size_t)blockIdx.x * hkv * row_bytes;
    for (int i = threadIdx.x; i < hkv * vec_per_row; i += blockDim.x) {
        const int g = i / vec_per_row, c = i - g * vec_per_row;
        const size_t src = src0 + (size_t)g * row_bytes + (size_t)c * 16;
        const size_t dst = (size_t)s * stride_scene_b + (size_t)g * stride_head_b + (size_t)row * stride_row_b + (size_t)c * 16;
        *reinterpret_cast<uint4*>(k + dst) = *reinterpret_cast<const uint4*>(k_new + src);
        *reinterpret_cast<uint4*>(v + dst) = *reinterpret_cast<const uint4*>(v_new + src);
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

extern "C" int fdc_kv_append(const fdc_plan* p, const fdc_kv_desc* kv, int32_t layer, const int32_t* d_n_active,
                             const int32_t* d_kv_row, const void* d_k_new, const void* d_v_new, void* stream)
{
    int rc = check_kv_desc(p, kv, layer);
    if (rc) return rc;
    if (!d_n_active || !d_kv_row || !d_k_new || !d_v_new) return FDC_ERR_NULL;
    if (((uintptr_t)d_k_new & 15) || ((uintptr_t)d_v_new & 15)) return FDC_ERR_SHAPE;
    const int es = kv->dtype == FDC_F32 ? 4 : 2;
    char* kb = (char*)kv->k + (size_t)layer * kv->stride_layer * es;
    char* vb = (char*)kv->v + (size_t)layer * kv->stride_layer * es;
    const int row_bytes = kv->head_dim * es;
    int threads = kv->hkv * (row_bytes >> 4);
    threads = threads > 256 ? 256 : ((threads + 31) & ~31);
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kv->batch * p->h.max_active);
        cfg.blockDim = dim3(threads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = (cudaStream_t)stream;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        FDC_CUDA(cudaLaunchKernelEx(&cfg, kv_append_kernel, kb, vb, (int64_t)(kv->stride_scene * es), (int64_t)(kv->stride_head * es),
                                    (int64_t)(kv->stride_row * es), (int)kv->rows, (int)kv->hkv, row_bytes, (int)p->h.max_active, d_n_active,
                                    d_kv_row, (const char*)d_k_new, (const char*)d_v_new, p->d_status));
    }
    note_launch();
    return FDC_OK;
}
