// The tcgen05 split-KV kernel, build for launches whose widest pair has up to 32 query rows (one
// group of softmax warps), and the entry points that choose between the builds.
#define FDC_TC_NGRP 1
#define FDC_TC_NPMAX 32
#define FDC_TC_KERNEL attn_tc_kernel
#define FDC_TC_LAUNCH launch_tc_np32
#define FDC_TC_TRACE_READ fdc_tr_read
#include "fdc_attn_tc_kernel.cuh"

namespace fdc {

int launch_tc_np64(const AttnParams& p, int head_dim, cudaStream_t st, int split_only);    // fdc_attn_tc_g2.cu
int launch_tc_np128(const AttnParams& p, int head_dim, cudaStream_t st, int split_only);   // fdc_attn_tc_w128.cu

static int launch_tc(const AttnParams& p, int head_dim, cudaStream_t st, int split_only)
{
    if (p.mmax > 64) return launch_tc_np128(p, head_dim, st, split_only);
    if (p.mmax > 32) return launch_tc_np64(p, head_dim, st, split_only);
    return launch_tc_np32(p, head_dim, st, split_only);
}

int launch_attn_tc(const AttnParams& p, int head_dim, cudaStream_t st) { return launch_tc(p, head_dim, st, 0); }
int launch_attn_tc_split(const AttnParams& p, int head_dim, cudaStream_t st) { return launch_tc(p, head_dim, st, 1); }

}  // namespace fdc
