// The tcgen05 split-KV kernel, build for launches whose widest pair has 65 to 128 query rows: one
// group of softmax warps, two score buffers and a single P^T buffer.
#define FDC_TC_NGRP 1
#define FDC_TC_NPMAX 128
#define FDC_TC_KERNEL attn_tc_kernel_w128
#define FDC_TC_LAUNCH launch_tc_np128
#define FDC_TC_TRACE_READ fdc_tr_read_w128
#include "fdc_attn_tc_kernel.cuh"
