// Split-KV pass for bf16 caches on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Sec. 3.3: the queries of all parallel fields of a scene, times the GQA heads of a KV head,
// share ONE read of the KV rows.  Here they form the (zero-padded) 128-row M side of two
// tcgen05 MMAs per 64-row KV tile: S = Q K^T (accumulator in TMEM, 64 columns, double
// buffered) and O += P V (accumulator in TMEM, head_dim columns).  One persistent CTA per SM:
//   warps 8, 10 TMA producers: K tiles and V tiles into two 128B-swizzled shared-memory rings
//               (a K stage is free again after its S = Q K^T, a V stage after its O += P V)
//   warp 9      MMA issuer (one elected thread), allocates / frees TMEM; S = Q K^T is issued up
//               to four tiles ahead of the softmax (four score buffers in TMEM)
//   warps 0-7   softmax.  A warp can only read the 32 TMEM lanes of its quadrant (warp % 4), so
//               when there are at most 32 (64) query rows they are replicated 4 (2) times along
//               M: every quadrant then holds a copy of each score row and the 8 warps split the
//               64 score columns of a row between them (8, 16 or 32 columns per thread).  Each
//               thread applies its branch's row bitmap (Eq. 1) by select, exponentiates against
//               the row's reference maximum and writes its slice of P (bf16) to shared memory,
//               the A operand of P V.
// The reference maximum of a row is shared by its threads and only raised when some slice
// maximum exceeds it by more than 2^8 (found with one barrier-wide OR per tile); the slices'
// maxima are then exchanged through shared memory and the accumulator row is rescaled in
// TMEM.  Results are exact either way: sum and accumulator use the same reference.
#include <cudaTypedefs.h>

#include "fdc_attn_common.cuh"

using namespace fdc;

namespace {

constexpr int TILE = FDC_TILE_ROWS;          // KV rows per tile = N of the QK MMA, K of the PV MMA
constexpr int MROWS = 128;                   // M of both MMAs (query rows, zero padded)
constexpr int NSOFT = 8;                     // softmax warps
constexpr int W_KPROD = 8, W_MMA = 9, W_VPROD = 10;
constexpr int THREADS = 352;
constexpr int NSBUF = 4;                     // score buffers in TMEM: S = Q K^T runs up to 4 tiles ahead
constexpr uint32_t TMEM_COLS = 512;          // S0..S3 [0,256) | O [256, 256 + head_dim)
constexpr int MAXRING = 8;                   // stages per ring (K ring, V ring)
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : FDC_R8(v, 0), FDC_R8(v, 8)
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];" : FDC_R8(v, 0) : "r"(taddr) : "memory");
}
template <int WS>
__device__ __forceinline__ void tmem_ld_slice(uint32_t taddr, uint32_t (&v)[32])
{
    if constexpr (WS == 32) tmem_ld32(taddr, v);
    else if constexpr (WS == 16) tmem_ld16(taddr, v);
    else tmem_ld8(taddr, v);
}
// OR of a predicate over the softmax threads (named barrier 1)
__device__ __forceinline__ bool soft_any(bool x)
{
    uint32_t out;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(out)
                 : "r"((uint32_t)x), "n"(NSOFT * 32)
                 : "memory");
    return out != 0;
}
__device__ __forceinline__ void soft_sync() { asm volatile("bar.sync 1, %0;" ::"n"(NSOFT * 32) : "memory"); }
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
    static constexpr int KV_BYTES = TILE * D * 2;             // one K (or V) tile = one ring stage
    static constexpr int Q_PANEL = MROWS * 128;
    static constexpr int Q_BYTES = MROWS * D * 2;
    static constexpr int P_BYTES = MROWS * TILE * 2;          // one P buffer: 128 rows x 128 bytes
};

// Everything a role needs to find its barriers and buffers.
struct Ctx {
    uint32_t k_full, k_empty, v_full, v_empty, s_full, p_full, pv_done, q_ready, o_free;
    uint32_t tm_s, tm_o;
    unsigned char *kring, *vring, *qs, *ps;
    float* xch;
    int* pre;
    volatile int* abortp;
    int nk, nv;
};

// One TMA producer warp: streams the K (or V) tiles of this CTA's units into its ring.
template <int D>
__device__ __forceinline__ void producer_loop(const AttnParams& p, const Ctx& cx, const CUtensorMap* tm, unsigned char* ring,
                                              uint32_t full, uint32_t empty, int nst, long long lo, long long hi, int lane)
{
    using L = Smem<D>;
    int s = 0;
    uint32_t it = 0;
    long long u = lo;
    int ok = 1;
    while (u < hi && ok) {
        const Segment sg = decode_segment(u, hi, cx.pre, p.hkv, s);
        for (int jb = sg.j0; jb < sg.j1 && ok; jb += 32) {
            const int jn = sg.j1 - jb < 32 ? sg.j1 - jb : 32;
            const int my_tile = lane < jn ? p.tiles[(size_t)sg.s * p.ntile_max + jb + lane] : 0;
            for (int k = 0; k < jn && ok; ++k, ++it) {
                const int tile = __shfl_sync(0xffffffffu, my_tile, k);
                if (lane == 0) {
                    const int st = it % nst;
                    if (!mbar_wait(empty + 8 * st, ((it / nst) & 1) ^ 1, cx.abortp, p.status)) {
                        ok = 0;
                    } else {
                        const uint32_t dst = smem_u32(ring + (size_t)st * L::KV_BYTES);
                        mbar_expect_tx(full + 8 * st, L::KV_BYTES);
#pragma unroll
                        for (int h = 0; h < D / 64; ++h)
                            tma_load_4d(dst + h * L::KV_PANEL, tm, full + 8 * st, h * 64, tile * TILE, sg.g, sg.s);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
            }
        }
        u = sg.next_u;
    }
    if (!ok && lane == 0) {
        // give the copies already in flight a bounded chance to land before the CTA ends
        const uint32_t first = it > (uint32_t)nst ? it - nst : 0;
        for (uint32_t k = first; k < it; ++k) {
            const uint32_t bar = full + 8 * (k % nst), ph = (k / nst) & 1;
            for (uint32_t i = 0; i < (1u << 16) && !mbar_try(bar, ph); ++i) __nanosleep(64);
        }
    }
}

// The MMA issuer thread.
template <int D>
__device__ __forceinline__ void mma_loop(const AttnParams& p, const Ctx& cx, long long lo, long long hi)
{
    using L = Smem<D>;
    const uint32_t idesc_qk = instr_desc(MROWS, TILE, 0), idesc_pv = instr_desc(MROWS, D, 1);
    const uint64_t q_desc = smem_desc(smem_u32(cx.qs), 16, 1024);
    const uint64_t p_desc = smem_desc(smem_u32(cx.ps), 16, 1024);
    const uint64_t k_desc0 = smem_desc(smem_u32(cx.kring), 16, 1024);
    const uint64_t v_desc0 = smem_desc(smem_u32(cx.vring), L::KV_PANEL, 1024);
    auto issue_qk = [&](uint32_t g) -> bool {
        const int st = g % cx.nk;
        if (!mbar_wait(cx.k_full + 8 * st, (g / cx.nk) & 1, cx.abortp, p.status)) return false;
        tc_fence_after();
        const uint64_t kd = k_desc0 + (uint64_t)((st * L::KV_BYTES) >> 4);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
            umma(cx.tm_s + (g & (NSBUF - 1)) * TILE, q_desc + (uint64_t)(((ks >> 2) * L::Q_PANEL + (ks & 3) * 32) >> 4),
                 kd + (uint64_t)(((ks >> 2) * L::KV_PANEL + (ks & 3) * 32) >> 4), idesc_qk, ks > 0);
        umma_commit(cx.k_empty + 8 * st);
        umma_commit(cx.s_full + 8 * (g & (NSBUF - 1)));
        return true;
    };
    int s = 0;
    uint32_t it = 0, seg = 0;
    long long u = lo;
    bool ok = true;
    while (u < hi && ok) {
        const Segment sg = decode_segment(u, hi, cx.pre, p.hkv, s);
        const int n = sg.j1 - sg.j0;
        ok = mbar_wait(cx.q_ready, seg & 1, cx.abortp, p.status);
        for (int a = 0; a < NSBUF && a < n && ok; ++a) ok = issue_qk(it + a);
        for (int t = 0; t < n && ok; ++t) {
            const uint32_t g = it + t;
            ok = mbar_wait(cx.p_full + 8 * (g & 1), (g >> 1) & 1, cx.abortp, p.status);
            if (ok && t == 0 && seg > 0) ok = mbar_wait(cx.o_free, (seg - 1) & 1, cx.abortp, p.status);
            const int st = g % cx.nv;
            if (ok) ok = mbar_wait(cx.v_full + 8 * st, (g / cx.nv) & 1, cx.abortp, p.status);
            if (!ok) break;
            tc_fence_after();
            const uint64_t vd = v_desc0 + (uint64_t)((st * L::KV_BYTES) >> 4);
            const uint64_t pd = p_desc + (uint64_t)(((g & 1) * L::P_BYTES) >> 4);
#pragma unroll
            for (int kk = 0; kk < TILE / 16; ++kk)
                umma(cx.tm_o, pd + (uint64_t)((kk * 32) >> 4), vd + (uint64_t)((kk * 2048) >> 4), idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
            umma_commit(cx.v_empty + 8 * st);
            umma_commit(cx.pv_done + 8 * (g & 1));
            if (t + NSBUF < n) ok = issue_qk(g + NSBUF);
        }
        it += n;
        ++seg;
        u = sg.next_u;
    }
}

// The softmax warps' work on one segment; WS = score columns per thread (64 / threads per row).
template <int D, int WS>
__device__ __forceinline__ void softmax_segment(const AttnParams& p, const Ctx& cx, const Segment& sg, uint32_t& it, bool& dead,
                                                const int warp, const int lane)
{
    using L = Smem<D>;
    constexpr int NSLICE = TILE / WS;             // threads sharing one query row
    constexpr int MP = MROWS * 2 / NSLICE;        // rows per replica
    const int q4 = warp & 3, half = warp >> 2;
    const int i_row = q4 * 32 + lane;             // MMA row = TMEM lane of this thread
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    const float c = p.scale_log2;
    const int A = p.n_active[sg.s];
    const int M = A * p.group;
    const int m = i_row & (MP - 1);               // query row of this thread
    const int sigma = (i_row / MP) * 2 + half;    // its column slice
    const int col0 = sigma * WS;
    const bool row_on = m < M;
    const bool warp_on = ((q4 * 32) & (MP - 1)) < M;      // some lane of the warp has a live row
    const bool owner = half == 0 && q4 * 32 < MP;         // warp whose TMEM lanes are the rows of replica 0
    const int br = row_on ? m / p.group : 0;
    const uint64_t* mrow = p.mask + ((size_t)sg.s * p.max_active + br) * p.W;
    auto wait_u = [&](uint32_t bar, uint32_t parity) {    // warp-uniform outcome
        if (!dead && !mbar_wait(bar, parity, cx.abortp, p.status)) dead = true;
        dead = __any_sync(0xffffffffu, dead);
    };
    // the query tile (A operand of S = Q K^T): MMA row i holds query row i mod MP; K-major, 128B swizzle
    if (!dead) {
        const uint4* src = reinterpret_cast<const uint4*>(
            reinterpret_cast<const __nv_bfloat16*>(p.q) +
            (((size_t)sg.s * p.max_active + br) * p.hq + (size_t)sg.g * p.group + (m - br * p.group)) * D);
#pragma unroll
        for (int cc = 0; cc < D / 16; ++cc) {
            const int ch = half * (D / 16) + cc;
            const uint4 v = row_on ? src[ch] : make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(cx.qs + (ch >> 3) * L::Q_PANEL + i_row * 128 + (((ch & 7) ^ (i_row & 7)) << 4)) = v;
        }
        fence_async_smem();
        mbar_arrive(cx.q_ready);
    }
    float ms = -INFINITY, l = 0.f;        // row reference maximum (scaled log2 units), this thread's partial sum
    const int n = sg.j1 - sg.j0;
    for (int jb = 0; jb < n; jb += 32) {
        const int jn = n - jb < 32 ? n - jb : 32;
        const int my_tile = lane < jn ? p.tiles[(size_t)sg.s * p.ntile_max + sg.j0 + jb + lane] : 0;
        for (int k = 0; k < jn; ++k, ++it) {
            const int tile = __shfl_sync(0xffffffffu, my_tile, k);
            const int t = jb + k;
            const uint32_t b = it & 1, sb = it & (NSBUF - 1);
            const bool masked = tile * TILE + TILE > p.P;
            wait_u(cx.s_full + 8 * sb, (it / NSBUF) & 1);
            tc_fence_after();
            if (masked && !dead) {
                // rows no branch may see can hold anything: clear their V so that 0 * NaN cannot arise
                wait_u(cx.v_full + 8 * (it % cx.nv), (it / cx.nv) & 1);
                uint64_t um = 0ull;
                for (int bb = lane; bb < A; bb += 32)
                    um |= tile_rowmask(p.mask + ((size_t)sg.s * p.max_active + bb) * p.W, p.W, p.P, tile);
                const uint32_t ul = __reduce_or_sync(0xffffffffu, (uint32_t)um);
                const uint32_t uh = __reduce_or_sync(0xffffffffu, (uint32_t)(um >> 32));
                uint64_t z = ~(((uint64_t)uh << 32) | ul);
                unsigned char* vs = cx.vring + (size_t)(it % cx.nv) * L::KV_BYTES;
                while (z && !dead) {
                    const int zr = __ffsll((long long)z) - 1;
                    z &= z - 1;
                    if ((zr & 7) != warp) continue;
                    for (int i = lane; i < D / 4; i += 32) {
                        const int ch = i >> 1;
                        *reinterpret_cast<uint2*>(vs + (ch >> 3) * L::KV_PANEL + zr * 128 + (((ch & 7) ^ (zr & 7)) << 4) + (i & 1) * 8) =
                            make_uint2(0u, 0u);
                    }
                }
            }
            uint32_t sv[32];
            float mx = -INFINITY;
            const bool work = warp_on && !dead;
            if (work) {
                tmem_ld_slice<WS>(cx.tm_s + lane_base + sb * TILE + col0, sv);
                tmem_wait_ld();
                uint32_t vis = row_on ? 0xffffffffu : 0u;
                if (masked && row_on) vis = (uint32_t)(tile_rowmask(mrow, p.W, p.P, tile) >> col0);
#pragma unroll
                for (int i = 0; i < WS; ++i) {
                    const float x = ((vis >> i) & 1) ? __uint_as_float(sv[i]) * c : -INFINITY;
                    sv[i] = __float_as_uint(x);
                    mx = fmaxf(mx, x);
                }
            }
            // does any row need a higher reference?  (first visible score, or a jump of more than 2^8)
            const bool flag = work && (ms == -INFINITY ? mx != -INFINITY : mx > ms + RESCALE_LOG2);
            if (soft_any(flag)) {
                cx.xch[m * NSLICE + sigma] = mx;
                soft_sync();
                float mr = -INFINITY;
#pragma unroll
                for (int j = 0; j < NSLICE; ++j) mr = fmaxf(mr, cx.xch[m * NSLICE + j]);
                const bool first = ms == -INFINITY && mr != -INFINITY;
                const bool jump = ms != -INFINITY && mr > ms + RESCALE_LOG2;
                const float alpha = jump ? fast_exp2(ms - mr) : 1.f;
                l *= alpha;
                if (owner && t > 0 && __any_sync(0xffffffffu, jump && work)) {
                    // O must not be written by an MMA while it is rescaled: the previous PV has to be complete
                    wait_u(cx.pv_done + 8 * ((it - 1) & 1), ((it - 1) >> 1) & 1);
                    tc_fence_after();
                    if (!dead) {
#pragma unroll
                        for (int cc = 0; cc < D / 32; ++cc) {
                            uint32_t ov[32];
                            tmem_ld32(cx.tm_o + lane_base + cc * 32, ov);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                            tmem_st32(cx.tm_o + lane_base + cc * 32, ov);
                        }
                        tmem_wait_st();
                    }
                }
                if (first || jump) ms = mr;
            }
            // P[b] is still being read until the PV of two tiles ago has completed
            wait_u(cx.pv_done + 8 * b, ((it >> 1) & 1) ^ 1);
            if (work && !dead) {
                const float mref = ms == -INFINITY ? 0.f : ms;
                unsigned char* prow = cx.ps + b * L::P_BYTES + m * 128;
#pragma unroll
                for (int ch = 0; ch < WS / 8; ++ch) {
                    float e[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) e[i] = fast_exp2(__uint_as_float(sv[ch * 8 + i]) - mref);
                    l += ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
                    *reinterpret_cast<uint4*>(prow + ((((col0 >> 3) + ch) ^ (m & 7)) << 4)) =
                        make_uint4(pack2(e[0], e[1]), pack2(e[2], e[3]), pack2(e[4], e[5]), pack2(e[6], e[7]));
                }
            }
            if (!dead) {
                tc_fence_before();
                fence_async_smem();
                mbar_arrive(cx.p_full + 8 * b);
            }
        }
    }
    // ---- end of segment: the accumulator is final once the last PV has completed
    const uint32_t last = it - 1;
    wait_u(cx.pv_done + 8 * (last & 1), (last >> 1) & 1);
    tc_fence_after();
    cx.xch[256 + m * NSLICE + sigma] = l;
    soft_sync();
    const int slot = blockIdx.x + sg.s * p.hkv + sg.g;
    if (owner && warp_on && !dead) {
        float lt = 0.f;
#pragma unroll
        for (int j = 0; j < NSLICE; ++j) lt += cx.xch[256 + m * NSLICE + j];
        float* wo = p.ws_o + ((size_t)slot * p.mmax + m) * D;
#pragma unroll
        for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t ov[32];
            tmem_ld32(cx.tm_o + lane_base + cc * 32, ov);
            tmem_wait_ld();
            if (row_on) {
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                    *reinterpret_cast<uint4*>(wo + cc * 32 + i) = make_uint4(ov[i], ov[i + 1], ov[i + 2], ov[i + 3]);
            }
        }
        if (row_on) *reinterpret_cast<float2*>(p.ws_ml + ((size_t)slot * p.mmax + m) * 2) = make_float2(ms, lt);
    }
    soft_sync();                     // the exchange buffer is free again
    if (!dead) {
        tc_fence_before();
        mbar_arrive(cx.o_free);
    }
}

template <int D>
__global__ void __launch_bounds__(THREADS, 1)
attn_tc_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const int nk, const int nv)
{
    using L = Smem<D>;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    Ctx cx;
    cx.nk = nk;
    cx.nv = nv;
    cx.kring = smem;
    cx.vring = cx.kring + (size_t)nk * L::KV_BYTES;
    cx.qs = cx.vring + (size_t)nv * L::KV_BYTES;
    cx.ps = cx.qs + L::Q_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(cx.ps + 2 * L::P_BYTES);
    cx.k_full = smem_u32(bars);
    cx.k_empty = cx.k_full + 8 * MAXRING;
    cx.v_full = cx.k_empty + 8 * MAXRING;
    cx.v_empty = cx.v_full + 8 * MAXRING;
    cx.s_full = cx.v_empty + 8 * MAXRING;
    cx.p_full = cx.s_full + 8 * NSBUF;
    cx.pv_done = cx.p_full + 16;
    cx.q_ready = cx.pv_done + 16;
    cx.o_free = cx.q_ready + 8;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 4 * MAXRING + NSBUF + 6);
    cx.xch = reinterpret_cast<float*>(tmem_holder + 2);      // [256] slice maxima, [256] slice sums
    cx.pre = reinterpret_cast<int*>(cx.xch + 512);
    __shared__ int abort_flag;
    cx.abortp = &abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) abort_flag = 0;
    const long long total = scan_ntiles(p.ntiles, p.batch, cx.pre);
    const long long U = total * p.hkv;
    if (U == 0) return;
    const long long lo = cta_first_unit(blockIdx.x, U, p.n_cta);
    const long long hi = cta_first_unit(blockIdx.x + 1, U, p.n_cta);
    if (lo >= hi) return;
    if (threadIdx.x == 0) {
        for (int i = 0; i < MAXRING; ++i) {
            mbar_init(cx.k_full + 8 * i, 1);
            mbar_init(cx.k_empty + 8 * i, 1);
            mbar_init(cx.v_full + 8 * i, 1);
            mbar_init(cx.v_empty + 8 * i, 1);
        }
        for (int i = 0; i < NSBUF; ++i) mbar_init(cx.s_full + 8 * i, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(cx.p_full + 8 * i, NSOFT * 32);
            mbar_init(cx.pv_done + 8 * i, 1);
        }
        mbar_init(cx.q_ready, NSOFT * 32);
        mbar_init(cx.o_free, NSOFT * 32);
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
    cx.tm_s = tmem;
    cx.tm_o = tmem + NSBUF * TILE;

    if (warp == W_KPROD) {
        producer_loop<D>(p, cx, &tm_k, cx.kring, cx.k_full, cx.k_empty, nk, lo, hi, lane);
    } else if (warp == W_VPROD) {
        producer_loop<D>(p, cx, &tm_v, cx.vring, cx.v_full, cx.v_empty, nv, lo, hi, lane);
    } else if (warp == W_MMA) {
        if (lane == 0) mma_loop<D>(p, cx, lo, hi);
    } else {
        int s = 0;
        uint32_t it = 0;
        long long u = lo;
        bool dead = false;                        // a bounded wait ran out somewhere in the CTA
        while (u < hi) {
            const Segment sg = decode_segment(u, hi, cx.pre, p.hkv, s);
            const int M = p.n_active[sg.s] * p.group;
            // at most 32 (64) query rows: replicated 4x (2x) along M, 8 (4) threads per row
            if (M <= 32) softmax_segment<D, 8>(p, cx, sg, it, dead, warp, lane);
            else if (M <= 64) softmax_segment<D, 16>(p, cx, sg, it, dead, warp, lane);
            else softmax_segment<D, 32>(p, cx, sg, it, dead, warp, lane);
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
    const size_t fixed = 1024 + L::Q_BYTES + 2 * L::P_BYTES + 8 * (4 * MAXRING + NSBUF + 6) + 16 + 2048 + sizeof(int) * (p.batch + 1) + 64;
    int stages = (int)((227 * 1024 - 256 - fixed) / L::KV_BYTES);
    if (stages > 2 * MAXRING) stages = 2 * MAXRING;
    if (stages < 4) return FDC_ERR_SHAPE;
    const int nk = stages / 2, nv = stages - nk;
    const size_t smem = fixed + (size_t)stages * L::KV_BYTES;
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
    attn_tc_kernel<D><<<p.n_cta, THREADS, smem, st>>>(p, tk, tv, nk, nv);
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
