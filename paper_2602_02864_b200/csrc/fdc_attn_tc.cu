// Split-KV pass for bf16 caches on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Sec. 3.3: the queries of all parallel fields of a scene, times the GQA heads of a KV head,
// share ONE read of the KV rows.  Here they form the (zero-padded) 128-row M side of two
// tcgen05 MMAs per 64-row KV tile: S = Q K^T (accumulator in TMEM, 64 columns, double
// buffered) and O += P V (accumulator in TMEM, head_dim columns).  One persistent CTA per SM:
//   warp 4      TMA producer: K and V tiles into a 128B-swizzled shared-memory ring
//   warp 5      MMA issuer (one elected thread), allocates / frees TMEM
//   warps 0-3   softmax: thread r owns query row r (TMEM lane r): loads its 64 scores,
//               applies its branch's row bitmap (Eq. 1) by select, keeps a running reference
//               maximum and sum, writes P (bf16) to shared memory as the A operand of P V
// The reference maximum is only raised when the new maximum exceeds it by more than 2^8
// (the accumulator then has to be rescaled in TMEM); results are exact either way because
// the same reference is used for the sum and the accumulator.
#include <cudaTypedefs.h>

#include "fdc_attn_common.cuh"

using namespace fdc;

namespace {

constexpr int TILE = FDC_TILE_ROWS;          // KV rows per tile = N of the QK MMA, K of the PV MMA
constexpr int MROWS = 128;                   // M of both MMAs (query rows, zero padded)
constexpr int W_PROD = 4, W_MMA = 5;
constexpr int THREADS = 192;
constexpr uint32_t TMEM_COLS = 256;          // S0 [0,64) | S1 [64,128) | O [128, 128 + head_dim)
constexpr float RESCALE_LOG2 = 8.f;

// ---------------------------------------------------------------- tcgen05 wrappers
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor (128-byte swizzle, descriptor version 1): start address,
// leading-dimension byte offset, stride-dimension byte offset, all in units of 16 bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulate, bf16 A and B, M x N, B optionally MN-major.
__device__ __forceinline__ uint32_t instr_desc(int m, int n, int b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

#define FDC_R8(v, o) "=r"(v[o + 0]), "=r"(v[o + 1]), "=r"(v[o + 2]), "=r"(v[o + 3]), "=r"(v[o + 4]), "=r"(v[o + 5]), "=r"(v[o + 6]), "=r"(v[o + 7])
#define FDC_I8(v, o) "r"(v[o + 0]), "r"(v[o + 1]), "r"(v[o + 2]), "r"(v[o + 3]), "r"(v[o + 4]), "r"(v[o + 5]), "r"(v[o + 6]), "r"(v[o + 7])
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,"
        "%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : FDC_R8(v, 0), FDC_R8(v, 8), FDC_R8(v, 16), FDC_R8(v, 24)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,"
        "%24,%25,%26,%27,%28,%29,%30,%31};"
        ::FDC_I8(v, 0), FDC_I8(v, 8), FDC_I8(v, 16), FDC_I8(v, 24), "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int D>
struct Smem {
    static constexpr int KV_PANEL = TILE * 128;               // 64 rows x 128 bytes
    static constexpr int KV_BYTES = TILE * D * 2;             // one K (or V) tile
    static constexpr int STAGE = 2 * KV_BYTES;
    static constexpr int Q_PANEL = MROWS * 128;
    static constexpr int Q_BYTES = MROWS * D * 2;
    static constexpr int P_BYTES = MROWS * TILE * 2;          // one P buffer: 128 rows x 128 bytes
};

template <int D>
__global__ void __launch_bounds__(THREADS, 1)
attn_tc_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const int nstage)
{
    using L = Smem<D>;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    unsigned char* stages = smem;
    unsigned char* qs = stages + (size_t)nstage * L::STAGE;
    unsigned char* ps = qs + L::Q_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ps + 2 * L::P_BYTES);
    // barrier indices
    const uint32_t kv_full = smem_u32(bars), kv_empty = kv_full + 8 * nstage;
    const uint32_t s_full = kv_empty + 8 * nstage, p_full = s_full + 16, pv_done = p_full + 16;
    const uint32_t q_ready = pv_done + 16, o_free = q_ready + 8;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * nstage + 8);
    int* pre = reinterpret_cast<int*>(tmem_holder + 2);
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) abort_flag = 0;
    const long long total = scan_ntiles(p.ntiles, p.batch, pre);
    const long long U = total * p.hkv;
    if (U == 0) return;
    const long long lo = cta_first_unit(blockIdx.x, U, p.n_cta);
    const long long hi = cta_first_unit(blockIdx.x + 1, U, p.n_cta);
    if (lo >= hi) return;
    if (threadIdx.x == 0) {
        for (int i = 0; i < nstage; ++i) {
            mbar_init(kv_full + 8 * i, 1);
            mbar_init(kv_empty + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s_full + 8 * i, 1);
            mbar_init(p_full + 8 * i, 128);
            mbar_init(pv_done + 8 * i, 1);
        }
        mbar_init(q_ready, 128);
        mbar_init(o_free, 128);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == W_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(tmem_holder);
    const uint32_t tm_s = tmem, tm_o = tmem + 2 * TILE;
    volatile int* abortp = &abort_flag;

    if (warp == W_PROD) {
        // ------------------------------------------------ TMA producer (lane 0 issues)
        int s = 0;
        uint32_t it = 0;
        long long u = lo;
        int ok = 1;
        while (u < hi && ok) {
            const Segment sg = decode_segment(u, hi, pre, p.hkv, s);
            for (int jb = sg.j0; jb < sg.j1 && ok; jb += 32) {
                const int jn = sg.j1 - jb < 32 ? sg.j1 - jb : 32;
                const int my_tile = lane < jn ? p.tiles[(size_t)sg.s * p.ntile_max + jb + lane] : 0;
                for (int k = 0; k < jn && ok; ++k, ++it) {
                    const int tile = __shfl_sync(0xffffffffu, my_tile, k);
                    if (lane == 0) {
                        const int st = it % nstage;
                        const uint32_t ph = (it / nstage) & 1;
                        if (!mbar_wait(kv_empty + 8 * st, ph ^ 1, abortp, p.status)) {
                            ok = 0;
                        } else {
                            const uint32_t dst = smem_u32(stages + (size_t)st * L::STAGE);
                            mbar_expect_tx(kv_full + 8 * st, L::STAGE);
#pragma unroll
                            for (int h = 0; h < D / 64; ++h) {
                                tma_load_4d(dst + h * L::KV_PANEL, &tm_k, kv_full + 8 * st, h * 64, tile * TILE, sg.g, sg.s);
                                tma_load_4d(dst + L::KV_BYTES + h * L::KV_PANEL, &tm_v, kv_full + 8 * st, h * 64, tile * TILE, sg.g, sg.s);
                            }
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                }
            }
            u = sg.next_u;
        }
        if (!ok && lane == 0) {
            const uint32_t first = it > (uint32_t)nstage ? it - nstage : 0;
            for (uint32_t k = first; k < it; ++k) {
                const uint32_t bar = kv_full + 8 * (k % nstage), ph = (k / nstage) & 1;
                for (uint32_t i = 0; i < (1u << 16) && !mbar_try(bar, ph); ++i) __nanosleep(64);
            }
        }
    } else if (warp == W_MMA) {
        // ------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            const uint32_t idesc_qk = instr_desc(MROWS, TILE, 0), idesc_pv = instr_desc(MROWS, D, 1);
            const uint32_t q_addr = smem_u32(qs), p_addr = smem_u32(ps);
            auto issue_qk = [&](uint32_t g) -> bool {
                const int st = g % nstage;
                if (!mbar_wait(kv_full + 8 * st, (g / nstage) & 1, abortp, p.status)) return false;
                tc_fence_after();
                const uint32_t k_addr = smem_u32(stages + (size_t)st * L::STAGE);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks & 3) * 32;
                    umma(tm_s + (g & 1) * TILE, smem_desc(q_addr + (ks >> 2) * L::Q_PANEL + off, 16, 1024),
                         smem_desc(k_addr + (ks >> 2) * L::KV_PANEL + off, 16, 1024), idesc_qk, ks > 0);
                }
                umma_commit(s_full + 8 * (g & 1));
                return true;
            };
            int s = 0;
            uint32_t it = 0, seg = 0;
            long long u = lo;
            bool ok = true;
            while (u < hi && ok) {
                const Segment sg = decode_segment(u, hi, pre, p.hkv, s);
                const int n = sg.j1 - sg.j0;
                ok = mbar_wait(q_ready, seg & 1, abortp, p.status);
                if (ok) ok = issue_qk(it);
                if (ok && n > 1) ok = issue_qk(it + 1);
                for (int t = 0; t < n && ok; ++t) {
                    const uint32_t g = it + t;
                    ok = mbar_wait(p_full + 8 * (g & 1), (g >> 1) & 1, abortp, p.status);
                    if (ok && t == 0 && seg > 0) ok = mbar_wait(o_free, (seg - 1) & 1, abortp, p.status);
                    if (!ok) break;
                    tc_fence_after();
                    const int st = g % nstage;
                    const uint32_t v_addr = smem_u32(stages + (size_t)st * L::STAGE) + L::KV_BYTES;
#pragma unroll
                    for (int kk = 0; kk < TILE / 16; ++kk)
                        umma(tm_o, smem_desc(p_addr + (g & 1) * L::P_BYTES + kk * 32, 16, 1024),
                             smem_desc(v_addr + kk * 2048, L::KV_PANEL, 1024), idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(kv_empty + 8 * st);
                    umma_commit(pv_done + 8 * (g & 1));
                    if (t + 2 < n) ok = issue_qk(g + 2);
                }
                it += n;
                ++seg;
                u = sg.next_u;
            }
        }
    } else {
        // ------------------------------------------------ softmax warps: thread r <-> query row r
        const int r = threadIdx.x;
        const float c = p.scale_log2;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const __nv_bfloat16* __restrict__ Qg = reinterpret_cast<const __nv_bfloat16*>(p.q);
        int s = 0;
        uint32_t it = 0;
        long long u = lo;
        bool ok = true;
        while (u < hi && ok) {
            const Segment sg = decode_segment(u, hi, pre, p.hkv, s);
            const int A = p.n_active[sg.s];
            const int M = A * p.group;
            const bool row_on = r < M, warp_on = warp * 32 < M;
            const int br = row_on ? r / p.group : 0;
            const uint64_t* mrow = p.mask + ((size_t)sg.s * p.max_active + br) * p.W;
            // the query tile (A operand of S = Q K^T): row r, K-major, 128-byte swizzle
            {
                const uint4* src = reinterpret_cast<const uint4*>(
                    Qg + (((size_t)sg.s * p.max_active + br) * p.hq + (size_t)sg.g * p.group + (r - br * p.group)) * D);
#pragma unroll
                for (int ch = 0; ch < D / 8; ++ch) {
                    const uint4 v = row_on ? src[ch] : make_uint4(0u, 0u, 0u, 0u);
                    *reinterpret_cast<uint4*>(qs + (ch >> 3) * L::Q_PANEL + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = v;
                }
                fence_async_smem();
                mbar_arrive(q_ready);
            }
            float ms = -INFINITY, l = 0.f;            // reference maximum (scaled log2 units) and running sum
            const int n = sg.j1 - sg.j0;
            for (int jb = 0; jb < n && ok; jb += 32) {
                const int jn = n - jb < 32 ? n - jb : 32;
                const int my_tile = lane < jn ? p.tiles[(size_t)sg.s * p.ntile_max + sg.j0 + jb + lane] : 0;
                for (int k = 0; k < jn && ok; ++k, ++it) {
                    const int tile = __shfl_sync(0xffffffffu, my_tile, k);
                    const int t = jb + k;
                    const uint32_t b = it & 1;
                    const int r0 = tile * TILE;
                    const bool masked = r0 + TILE > p.P;
                    if (!mbar_wait(s_full + 8 * b, (it >> 1) & 1, abortp, p.status)) { ok = false; break; }
                    tc_fence_after();
                    if (masked) {
                        // rows no branch may see can hold anything: clear their V so that 0 * NaN cannot arise
                        uint64_t um = 0ull;
                        for (int bb = lane; bb < A; bb += 32)
                            um |= tile_rowmask(p.mask + ((size_t)sg.s * p.max_active + bb) * p.W, p.W, p.P, tile);
                        const uint32_t ul = __reduce_or_sync(0xffffffffu, (uint32_t)um);
                        const uint32_t uh = __reduce_or_sync(0xffffffffu, (uint32_t)(um >> 32));
                        uint64_t z = ~(((uint64_t)uh << 32) | ul);
                        unsigned char* vs = stages + (size_t)(it % nstage) * L::STAGE + L::KV_BYTES;
                        while (z) {
                            const int zr = __ffsll((long long)z) - 1;
                            z &= z - 1;
                            if ((zr & 3) != warp) continue;
                            for (int i = lane; i < D / 4; i += 32) {
                                const int ch = i >> 1;
                                *reinterpret_cast<uint2*>(vs + (ch >> 3) * L::KV_PANEL + zr * 128 + (((ch & 7) ^ (zr & 7)) << 4) + (i & 1) * 8) =
                                    make_uint2(0u, 0u);
                            }
                        }
                    }
                    if (warp_on) {
                        uint32_t sv[2][32];
                        tmem_ld32(tm_s + lane_base + b * TILE, sv[0]);
                        tmem_ld32(tm_s + lane_base + b * TILE + 32, sv[1]);
                        tmem_wait_ld();
                        uint64_t vis = row_on ? ~0ull : 0ull;
                        if (masked && row_on) vis = tile_rowmask(mrow, p.W, p.P, tile);
                        float mx = -INFINITY;
#pragma unroll
                        for (int h = 0; h < 2; ++h)
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const float x = ((vis >> (h * 32 + i)) & 1) ? __uint_as_float(sv[h][i]) * c : -INFINITY;
                                sv[h][i] = __float_as_uint(x);
                                mx = fmaxf(mx, x);
                            }
                        // raise the reference only when needed: first visible score, or a jump of more than 2^8
                        const bool first = ms == -INFINITY && mx != -INFINITY;
                        const bool jump = ms != -INFINITY && mx > ms + RESCALE_LOG2;
                        if (__any_sync(0xffffffffu, jump)) {
                            // O must not be written by an MMA while it is rescaled: the previous PV has to be complete
                            if (t > 0 && !mbar_wait(pv_done + 8 * ((it - 1) & 1), ((it - 1) >> 1) & 1, abortp, p.status)) { ok = false; break; }
                            tc_fence_after();
                            const float alpha = jump ? fast_exp2(ms - mx) : 1.f;
                            l *= alpha;
                            if (t > 0) {
#pragma unroll
                                for (int cc = 0; cc < D / 32; ++cc) {
                                    uint32_t ov[32];
                                    tmem_ld32(tm_o + lane_base + cc * 32, ov);
                                    tmem_wait_ld();
#pragma unroll
                                    for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                                    tmem_st32(tm_o + lane_base + cc * 32, ov);
                                }
                                tmem_wait_st();
                            }
                        }
                        if (first || jump) ms = mx;
                        const float mref = ms == -INFINITY ? 0.f : ms;
                        // P[b] is still being read until the PV of two tiles ago has completed
                        if (!mbar_wait(pv_done + 8 * b, ((it >> 1) & 1) ^ 1, abortp, p.status)) { ok = false; break; }
                        unsigned char* prow = ps + b * L::P_BYTES + r * 128;
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch) {
                            float e[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                e[i] = fast_exp2(__uint_as_float(sv[ch >> 2][(ch & 3) * 8 + i]) - mref);
                                l += e[i];
                            }
                            *reinterpret_cast<uint4*>(prow + ((ch ^ (r & 7)) << 4)) =
                                make_uint4(pack2(e[0], e[1]), pack2(e[2], e[3]), pack2(e[4], e[5]), pack2(e[6], e[7]));
                        }
                    }
                    tc_fence_before();
                    fence_async_smem();
                    mbar_arrive(p_full + 8 * b);
                }
            }
            if (!ok) break;
            // ---- end of segment: the accumulator is final once the last PV has completed
            {
                const uint32_t last = it - 1;
                if (!mbar_wait(pv_done + 8 * (last & 1), (last >> 1) & 1, abortp, p.status)) { ok = false; break; }
                tc_fence_after();
                const int slot = blockIdx.x + sg.s * p.hkv + sg.g;
                if (warp_on) {
                    float* wo = p.ws_o + ((size_t)slot * p.mmax + r) * D;
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t ov[32];
                        tmem_ld32(tm_o + lane_base + cc * 32, ov);
                        tmem_wait_ld();
                        if (row_on) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4)
                                *reinterpret_cast<uint4*>(wo + cc * 32 + i) = make_uint4(ov[i], ov[i + 1], ov[i + 2], ov[i + 3]);
                        }
                    }
                    if (row_on) *reinterpret_cast<float2*>(p.ws_ml + ((size_t)slot * p.mmax + r) * 2) = make_float2(ms, l);
                }
                tc_fence_before();
                mbar_arrive(o_free);
            }
            u = sg.next_u;
        }
    }
    // ---- teardown: everybody is done with TMEM before it is freed
    tc_fence_before();
    __syncthreads();
    if (warp == W_MMA) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

template <int D>
int launch_t(const AttnParams& p, cudaStream_t st)
{
    using L = Smem<D>;
    const size_t fixed = 1024 + L::Q_BYTES + 2 * L::P_BYTES + 8 * (2 * 8 + 8) + 16 + sizeof(int) * (p.batch + 1) + 64;
    int nstage = (int)((227 * 1024 - 256 - fixed) / L::STAGE);
    if (nstage > 8) nstage = 8;
    if (nstage < 2) return FDC_ERR_SHAPE;
    const size_t smem = fixed + (size_t)nstage * L::STAGE;
    static size_t attr_smem = 0;
    if (smem > attr_smem) {
        cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return set_cuda_error(e);
        attr_smem = smem;
    }
    alignas(64) CUtensorMap tk, tv;
    int rc = get_kv_tensor_map(p.k, p, D, TILE, &tk);
    if (rc) return rc;
    rc = get_kv_tensor_map(p.v, p, D, TILE, &tv);
    if (rc) return rc;
    attn_tc_kernel<D><<<p.n_cta, THREADS, smem, st>>>(p, tk, tv, nstage);
    note_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FDC_OK : set_cuda_error(e);
}

}  // namespace

namespace fdc {

// bf16 only, at most 128 query rows per (scene, KV head).
int launch_attn_tc(const AttnParams& p, int head_dim, cudaStream_t st)
{
    return head_dim == 64 ? launch_t<64>(p, st) : launch_t<128>(p, st);
}

}  // namespace fdc
