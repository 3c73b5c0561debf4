// The tcgen05 split-KV kernel, build for one group of softmax warps (launches whose widest pair
// has up to 32 or more than 64 query rows), and the entry points that choose between the builds.
#define FDC_TC_NGRP 1
#define FDC_TC_KERNEL attn_tc_kernel
#define FDC_TC_LAUNCH launch_tc_one_group
#define FDC_TC_TRACE_READ fdc_tr_read
#include "fdc_attn_tc_kernel.cuh"

namespace fdc {

int launch_tc_two_groups(const AttnParams& p, int head_dim, cudaStream_t st, int split_only);   // fdc_attn_tc_g2.cu

static int launch_tc(const AttnParams& p, int head_dim, cudaStream_t st, int split_only)
{
    return (p.mmax > 32 && p.mmax <= 64) ? launch_tc_two_groups(p, head_dim, st, split_only)
                                         : launch_tc_one_group(p, head_dim, st, split_only);
}

int launch_attn_tc(const AttnParams& p, int head_dim, cudaStream_t st) { return launch_tc(p, head_dim, st, 0); }
int launch_attn_tc_split(const AttnParams& p, int head_dim, cudaStream_t st) { return launch_tc(p, head_dim, st, 1); }

}  // namespace fdc
