// fdc_selftest_bounded_wait: runs the bounded mbarrier wait that every TMA kernel of the library
// relies on against a barrier that nothing will ever complete, so that the limit itself can be
// exercised on a GPU: the wait must end on its own, report FDC_DEV_TIMEOUT through the plan's
// status word, and leave the context usable.
#include "fdc_attn_common.cuh"

using namespace fdc;

namespace {

__global__ void bounded_wait_kernel(int32_t* status, int32_t* outcome)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);                    // one arrival expected; none will come
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // all threads wait like the kernels' warps do: the first to reach the limit raises the CTA's abort
    // flag and the others leave on seeing it
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status);
    const int gave_up = __syncthreads_count(!ok);
    if (threadIdx.x == 0) *outcome = gave_up;
}

}  // namespace

extern "C" int fdc_selftest_bounded_wait(fdc_plan* p, int32_t* d_outcome, void* stream)
{
    if (!p || !d_outcome) return FDC_ERR_NULL;
    {
        int rcf = flush_pending_append(p);
        if (rcf) return rcf;
    }
    bounded_wait_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(p->d_status, d_outcome);
    note_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FDC_OK : set_cuda_error(e);
}
