// Device helpers shared by the TMA-fed split-KV kernels (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>

#include "fdc_internal.h"

namespace fdc {

constexpr uint32_t SPIN_LIMIT = 1u << 18;      // polls of a bounded wait: about a second (a poll that finds the phase incomplete is suspended for a few microseconds by the hardware)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after SPIN_LIMIT polls (or when another thread of the CTA gave up),
// records FDC_DEV_TIMEOUT and returns false; the caller then skips all further work.  The
// polling loop is kept out of line: most waits are already satisfied when they are reached,
// and the callers' loops stay small.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status)
{
    for (uint32_t i = 0; i < SPIN_LIMIT; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 255u) == 255u) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    *abort_flag = 1;
    atomicOr(status, 8 /* FDC_DEV_TIMEOUT */);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status)
{
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status);
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
// The same copy with an L2 eviction priority (a policy made by l2_evict_first_policy).
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
        : "memory");
}
// Lines read under this policy are the first to leave L2: for data that is read once (the KV
// stream), so that it does not push out what is read again (queries, bitmaps, tile lists,
// partial results, the kernel's own code).
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Exclusive prefix sums of ntiles over scenes into smem pre[0..batch]; returns the total.
// Called by every thread of the CTA (contains a __syncthreads()).
__device__ __forceinline__ int scan_ntiles(const int32_t* __restrict__ ntiles, int batch, int* pre)
{
    if (threadIdx.x < 32) {
        int carry = 0;
        for (int b0 = 0; b0 < batch; b0 += 32) {
            int i = b0 + threadIdx.x;
            int x = i < batch ? ntiles[i] : 0;
            int inc = x;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int y = __shfl_up_sync(0xffffffffu, inc, o);
                if ((int)threadIdx.x >= o) inc += y;
            }
            if (i < batch) pre[i] = carry + inc - x;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (threadIdx.x == 0) pre[batch] = carry;
    }
    __syncthreads();
    return pre[batch];
}

struct Segment {
    int s, g, j0, j1, nt;
    long long next_u;
};
// The run of units starting at u that belongs to one (scene, KV head) pair, cut at `hi`.
__device__ __forceinline__ Segment decode_segment(long long u, long long hi, const int* pre, int hkv, int& s)
{
    while ((long long)pre[s + 1] * hkv <= u) ++s;
    Segment sg;
    sg.s = s;
    sg.nt = pre[s + 1] - pre[s];
    const long long u_scene = (long long)pre[s] * hkv;
    sg.g = (int)((u - u_scene) / sg.nt);
    const long long pair0 = u_scene + (long long)sg.g * sg.nt;
    sg.j0 = (int)(u - pair0);
    const long long end = pair0 + sg.nt < hi ? pair0 + sg.nt : hi;
    sg.j1 = (int)(end - pair0);
    sg.next_u = end;
    return sg;
}


// Host: a cached 4-D tensor map (head_dim, rows, hkv, batch) of a bf16 cache with boxes of
// 64 elements x box_rows rows and 128-byte swizzle.  out_map points to a CUtensorMap.
int get_kv_tensor_map(const void* base, const AttnParams& p, int head_dim, int box_rows, void* out_map);

}  // namespace fdc
