// The tcgen05 split-KV kernel, build for launches whose widest pair has 33 to 64 query rows: two
// groups of softmax warps on alternate rounds.
#define FDC_TC_NGRP 2
#define FDC_TC_NPMAX 64
#define FDC_TC_KERNEL attn_tc_kernel_g2
#define FDC_TC_LAUNCH launch_tc_np64
#define FDC_TC_TRACE_READ fdc_tr_read_g2
#include "fdc_attn_tc_kernel.cuh"
