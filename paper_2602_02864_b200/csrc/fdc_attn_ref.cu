// Reference split-KV kernel on CUDA cores (any dtype, exact fp32 arithmetic) and the combine
// pass.  Sec. 3.3: every visited KV tile of a (scene, KV head) pair is read once and serves
// all branches and all GQA heads of that pair; the per-branch bitmap selects what each query
// row may see.  Used for the fp32 configuration and as the fallback for every other one.
#include <cuda_bf16.h>

#include "fdc_attn_common.cuh"

using namespace fdc;

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_max(float x)
{
#pragma unroll
    for (int o = 16; o; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads, 1) attn_ref_kernel(const AttnParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int KS = D + 1;                       // padded K row stride (conflict-free row-per-lane reads)
    float* Ks = reinterpret_cast<float*>(smem_raw);              // [64][D+1]
    float* Vs = Ks + 64 * KS;                                    // [64][D]
    float* Qs = Vs + 64 * D;                                     // [mmax][D]
    float* Os = Qs + (size_t)p.mmax * D;                         // [mmax][D]
    float* Ps = Os + (size_t)p.mmax * D;                         // [warps][64]
    float* ms = Ps + kWarps * 64;                                // [mmax]
    float* ls = ms + p.mmax;                                     // [mmax]
    int* pre = reinterpret_cast<int*>(ls + p.mmax);              // [batch+1]

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long total = scan_ntiles(p.ntiles, p.batch, pre);
    const long long U = total * p.hkv;
    if (U == 0) return;
    const long long lo = cta_first_unit(blockIdx.x, U, p.n_cta);
    const long long hi = cta_first_unit(blockIdx.x + 1, U, p.n_cta);
    const T* __restrict__ Kg = reinterpret_cast<const T*>(p.k);
    const T* __restrict__ Vg = reinterpret_cast<const T*>(p.v);
    const T* __restrict__ Qg = reinterpret_cast<const T*>(p.q);

    long long u = lo;
    int s = 0;
    while (u < hi) {
        while ((long long)pre[s + 1] * p.hkv <= u) ++s;          // scene holding unit u
        const int nt = pre[s + 1] - pre[s];
        const long long u_scene = (long long)pre[s] * p.hkv;
        const int g = (int)((u - u_scene) / nt);
        const int j0 = (int)((u - u_scene) - (long long)g * nt);
        const long long seg_end_ll = u_scene + (long long)(g + 1) * nt;
        const int j1 = (int)((hi < seg_end_ll ? hi : seg_end_ll) - u_scene - (long long)g * nt);
        const int A = p.n_active[s];
        const int M = A * p.group;
        const int slot = blockIdx.x + s * p.hkv + g;

        // queries of this (scene, KV head): row m = branch * group + head-in-group
        for (int i = threadIdx.x; i < M * D; i += kThreads) {
            int m = i / D, d = i - m * D;
            int b = m / p.group, hg = m - b * p.group;
            size_t qo = (((size_t)s * p.max_active + b) * p.hq + (size_t)g * p.group + hg) * D + d;
            Qs[i] = to_f32<T>(Qg[qo]) * p.scale_log2;
            Os[i] = 0.f;
        }
        for (int m = threadIdx.x; m < M; m += kThreads) {
            ms[m] = -INFINITY;
            ls[m] = 0.f;
        }
        const size_t kv_base = (size_t)s * p.stride_scene + (size_t)g * p.stride_head;
        for (int j = j0; j < j1; ++j) {
            const int tile = p.tiles[(size_t)s * p.ntile_max + j];
            const int r0 = tile * FDC_TILE_ROWS;
            __syncthreads();
            // stage the tile as fp32 (rows past the end of the cache read as zero)
            constexpr int VEC = 16 / sizeof(T);
            for (int i = threadIdx.x; i < 64 * (D / VEC); i += kThreads) {
                const int r = i / (D / VEC), c = (i - r * (D / VEC)) * VEC;
                float kf[VEC], vf[VEC];
                if (r0 + r < p.rows) {
                    const size_t off = kv_base + (size_t)(r0 + r) * p.stride_row + c;
                    uint4 kk = *reinterpret_cast<const uint4*>(Kg + off);
                    uint4 vv = *reinterpret_cast<const uint4*>(Vg + off);
                    const T* kp = reinterpret_cast<const T*>(&kk);
                    const T* vp = reinterpret_cast<const T*>(&vv);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        kf[e] = to_f32<T>(kp[e]);
                        vf[e] = to_f32<T>(vp[e]);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) kf[e] = vf[e] = 0.f;
                }
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    Ks[r * KS + c + e] = kf[e];
                    Vs[r * D + c + e] = vf[e];
                }
            }
            __syncthreads();
            for (int m = warp; m < M; m += kWarps) {
                const int b = m / p.group;
                uint64_t rm = tile_rowmask(p.mask + ((size_t)s * p.max_active + b) * p.W, p.W, p.P, tile);
                if (p.rows - r0 < 64) rm &= (1ull << (p.rows - r0)) - 1ull;
                if (rm == 0ull) continue;
                const bool on0 = (rm >> lane) & 1, on1 = (rm >> (lane + 32)) & 1;
                float s0 = 0.f, s1 = 0.f;
                const float* qrow = Qs + (size_t)m * D;
                const float* k0 = Ks + lane * KS;
                const float* k1 = Ks + (lane + 32) * KS;
#pragma unroll 8
                for (int d = 0; d < D; ++d) {
                    const float qd = qrow[d];
                    s0 = fmaf(qd, k0[d], s0);
                    s1 = fmaf(qd, k1[d], s1);
                }
                s0 = on0 ? s0 : -INFINITY;
                s1 = on1 ? s1 : -INFINITY;
                const float m_old = ms[m];
                const float m_new = fmaxf(m_old, warp_max(fmaxf(s0, s1)));   // finite: rm != 0
                const float alpha = exp2f(m_old - m_new);                    // m_old = -inf -> 0
                const float p0 = on0 ? exp2f(s0 - m_new) : 0.f;
                const float p1 = on1 ? exp2f(s1 - m_new) : 0.f;
                const float psum = warp_sum(p0 + p1);
                Ps[warp * 64 + lane] = p0;
                Ps[warp * 64 + lane + 32] = p1;
                __syncwarp();
                if (lane == 0) {
                    ms[m] = m_new;
                    ls[m] = ls[m] * alpha + psum;
                }
#pragma unroll
                for (int d = lane; d < D; d += 32) {
                    float acc = Os[(size_t)m * D + d] * alpha;
                    uint64_t bits = rm;
                    while (bits) {                       // only visible rows: an invisible V row may be NaN
                        const int r = __ffsll((long long)bits) - 1;
                        bits &= bits - 1;
                        acc = fmaf(Ps[warp * 64 + r], Vs[r * D + d], acc);
                    }
                    Os[(size_t)m * D + d] = acc;
                }
                __syncwarp();
            }
        }
        __syncthreads();
        // partial (m, l, O) of this segment
        float* wo = p.ws_o + (size_t)slot * p.mmax * D;
        float* wml = p.ws_ml + (size_t)slot * p.mmax * 2;
        for (int i = threadIdx.x; i < M * D; i += kThreads) wo[i] = Os[i];
        for (int m = threadIdx.x; m < M; m += kThreads) {
            wml[2 * m] = ms[m];
            wml[2 * m + 1] = ls[m];
        }
        __syncthreads();
        u = u_scene + (long long)g * nt + j1;
    }
}

// One warp per (scene, branch, query head): merge the partials of the CTAs that covered the
// pair's tiles.  m = max_j m_j; l = sum_j l_j 2^(m_j - m); O = sum_j O_j 2^(m_j - m) / l.
template <typename T, int D>
__global__ void __launch_bounds__(128) attn_combine_kernel(const AttnParams p)
{
    const int lane = threadIdx.x & 31;
    const int wid = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int per_scene = p.max_active * p.hq;
    if (wid >= p.batch * per_scene) return;
    const int s = wid / per_scene;
    const int rem = wid - s * per_scene;
    const int b = rem / p.hq, h = rem - b * p.hq;
    if (b >= p.n_active[s]) return;
    const int nt = p.ntiles[s];
    if (nt == 0) return;
    // tiles before this scene and in total (warp-strided sums)
    long long before = 0, total = 0;
    for (int i = lane; i < p.batch; i += 32) {
        int x = p.ntiles[i];
        total += x;
        if (i < s) before += x;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    const long long U = total * p.hkv;
    const int g = h / p.group, hg = h - g * p.group;
    const long long u0 = before * p.hkv + (long long)g * nt;
    const int c_first = unit_cta(u0, U, p.n_cta), c_last = unit_cta(u0 + nt - 1, U, p.n_cta);
    const int pair = s * p.hkv + g;
    const int m = b * p.group + hg;
    float mx = -INFINITY;
    // CTAs between the first and the last may own no unit at all (fewer units than CTAs)
    for (int c = c_first; c <= c_last; ++c) {
        if (cta_first_unit(c, U, p.n_cta) >= cta_first_unit(c + 1, U, p.n_cta)) continue;
        mx = fmaxf(mx, p.ws_ml[((size_t)(c + pair) * p.mmax + m) * 2]);
    }
    float l = 0.f;
    float acc[D / 32];
#pragma unroll
    for (int i = 0; i < D / 32; ++i) acc[i] = 0.f;
    for (int c = c_first; c <= c_last; ++c) {
        if (cta_first_unit(c, U, p.n_cta) >= cta_first_unit(c + 1, U, p.n_cta)) continue;
        const size_t slot = (size_t)(c + pair);
        const float mj = p.ws_ml[(slot * p.mmax + m) * 2];
        const float lj = p.ws_ml[(slot * p.mmax + m) * 2 + 1];
        const float w = exp2f(mj - mx);                  // a split that saw nothing: mj = -inf -> 0
        l = fmaf(lj, w, l);
        const float* o = p.ws_o + (slot * p.mmax + m) * D;
#pragma unroll
        for (int i = 0; i < D / 32; ++i) acc[i] = fmaf(o[lane + 32 * i], w, acc[i]);
    }
    const float inv = 1.f / l;
    T* out = reinterpret_cast<T*>(p.out) + (((size_t)s * p.max_active + b) * p.hq + h) * D;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) out[lane + 32 * i] = from_f32<T>(acc[i] * inv);
}

template <typename T, int D>
int launch_ref_t(const AttnParams& p, cudaStream_t st)
{
    size_t smem = sizeof(float) * ((size_t)64 * (D + 1) + 64 * D + 2 * (size_t)p.mmax * D + kWarps * 64 + 2 * p.mmax) +
                  sizeof(int) * (p.batch + 1);
    if (smem > 227 * 1024) return FDC_ERR_SHAPE;
    static size_t attr_smem[kMaxDevices] = {};
    const int rcs = raise_dynamic_smem(reinterpret_cast<const void*>(attn_ref_kernel<T, D>), smem, attr_smem);
    if (rcs) return rcs;
    attn_ref_kernel<T, D><<<p.n_cta, kThreads, smem, st>>>(p);
    note_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FDC_OK : set_cuda_error(e);
}

template <typename T, int D>
int launch_combine_t(const AttnParams& p, cudaStream_t st)
{
    const int warps = p.batch * p.max_active * p.hq;
    attn_combine_kernel<T, D><<<(warps + 3) / 4, 128, 0, st>>>(p);
    note_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FDC_OK : set_cuda_error(e);
}

}  // namespace

namespace fdc {

int launch_attn_ref(const AttnParams& p, int dtype, int head_dim, cudaStream_t st)
{
    if (dtype == FDC_F32) return head_dim == 64 ? launch_ref_t<float, 64>(p, st) : launch_ref_t<float, 128>(p, st);
    return head_dim == 64 ? launch_ref_t<__nv_bfloat16, 64>(p, st) : launch_ref_t<__nv_bfloat16, 128>(p, st);
}

int launch_attn_combine(const AttnParams& p, int dtype, int head_dim, cudaStream_t st)
{
    if (dtype == FDC_F32) return head_dim == 64 ? launch_combine_t<float, 64>(p, st) : launch_combine_t<float, 128>(p, st);
    return head_dim == 64 ? launch_combine_t<__nv_bfloat16, 64>(p, st) : launch_combine_t<__nv_bfloat16, 128>(p, st);
}

}  // namespace fdc
