// Split-KV pass for bf16 caches: TMA-fed shared-memory ring + tensor-core MMA.
//
// Sec. 3.3: all queries decoded in one forward pass (one per parallel field, times the GQA
// heads of a KV head) share ONE read of the scene's KV rows.  Here a persistent CTA per SM
// streams its share of the visited 64-row KV tiles, as 32-row half tiles, through a ring of
// TMA-filled, 128B-swizzled shared-memory stages; 8 consumer warps hold the query rows as MMA
// A fragments (16-row blocks) and run an online softmax (running max / sum, fp32) per row.
// When there are fewer 16-row query blocks than warps, the warps form several "KV lanes":
// lane k takes every k-th stage for itself (whole stage: long independent MMA chains), and
// the lanes' partial results are merged at the end of a segment.  The per-branch row bitmaps (Eq. 1) are
// applied by select on the scores; tiles wholly inside the prefix skip masking.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cudaTypedefs.h>

#include <mutex>
#include <vector>

#include "fdc_attn_common.cuh"

using namespace fdc;

namespace {

constexpr int NW = 8;                    // consumer warps
constexpr int THREADS = (NW + 1) * 32;   // + 1 producer warp
constexpr int TILE = FDC_TILE_ROWS;
constexpr int SROWS = 32;                // KV rows per shared-memory stage (half a tile)
constexpr int HALVES = TILE / SROWS;     // stages per tile

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory"); }

// Byte offset of the 16-byte chunk `dc` (0 .. D/8-1) of row `r` inside a K or V tile staged by
// TMA with 128-byte swizzle: the stage holds D/64 panels of [SROWS rows][128 bytes]; inside a
// panel the chunk index is XORed with (row mod 8).
__device__ __forceinline__ uint32_t tile_off(int r, int dc)
{
    return (uint32_t)((dc >> 3) * (SROWS * 128) + r * 128 + (((dc & 7) ^ (r & 7)) << 4));
}

// One staged half tile (SROWS rows) for one consumer warp.
template <int D>
__device__ __forceinline__ void process_stage(const uint32_t kbase, const uint32_t vbase, unsigned char* vgen,
                                              const uint32_t (&qf)[D / 16][4], float (&o)[D / 8][4], float& m_lo, float& m_hi,
                                              float& l_lo, float& l_hi, const bool masked, const uint64_t mk_lo,
                                              const uint64_t mk_hi, const uint64_t zero_rows, const float c, const int lane)
{
    constexpr int NT = SROWS / 8;
    float sacc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
    // S = Q K^T: NT independent accumulator chains
#pragma unroll
    for (int ks = 0; ks < D / 16; ks += 2) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int r = nt * 8 + (lane & 7);
            uint32_t b0, b1, b2, b3;
            ldsm_x4(kbase + tile_off(r, 2 * ks + (lane >> 3)), b0, b1, b2, b3);
            mma_bf16(sacc[nt], qf[ks], b0, b1);
            mma_bf16(sacc[nt], qf[ks + 1], b2, b3);
        }
    }
    if (masked) {
        // rows nobody may see can hold anything: clear their V so that 0 * NaN cannot arise
        uint64_t z = zero_rows;
        while (z) {
            const int r = __ffsll((long long)z) - 1;
            z &= z - 1;
            for (int i = lane; i < D / 4; i += 32)        // D*2 bytes = D/4 words of 8 bytes
                *reinterpret_cast<uint2*>(vgen + tile_off(r, i >> 1) + (i & 1) * 8) = make_uint2(0u, 0u);
        }
        __syncwarp();
        const int cb = 2 * (lane & 3);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int col = nt * 8 + cb;
            if (!((mk_lo >> col) & 1)) sacc[nt][0] = -INFINITY;
            if (!((mk_lo >> (col + 1)) & 1)) sacc[nt][1] = -INFINITY;
            if (!((mk_hi >> col) & 1)) sacc[nt][2] = -INFINITY;
            if (!((mk_hi >> (col + 1)) & 1)) sacc[nt][3] = -INFINITY;
        }
    }
    // online softmax (scores in raw units; c = scale * log2 e is folded into the exponent)
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        mx_lo = fmaxf(mx_lo, fmaxf(sacc[nt][0], sacc[nt][1]));
        mx_hi = fmaxf(mx_hi, fmaxf(sacc[nt][2], sacc[nt][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float ms_lo = mn_lo == -INFINITY ? 0.f : mn_lo * c;      // a row that has seen nothing yet
    const float ms_hi = mn_hi == -INFINITY ? 0.f : mn_hi * c;
    // the running maxima settle after a few tiles: rescale only when one of them moved
    const bool moved = (mn_lo != m_lo) || (mn_hi != m_hi);
    if (__any_sync(0xffffffffu, moved)) {
        const float a_lo = fast_exp2(m_lo * c - ms_lo), a_hi = fast_exp2(m_hi * c - ms_hi);
        l_lo *= a_lo;
        l_hi *= a_hi;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            o[i][0] *= a_lo;
            o[i][1] *= a_lo;
            o[i][2] *= a_hi;
            o[i][3] *= a_hi;
        }
        m_lo = mn_lo;
        m_hi = mn_hi;
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        sacc[nt][0] = fast_exp2(fmaf(sacc[nt][0], c, -ms_lo));
        sacc[nt][1] = fast_exp2(fmaf(sacc[nt][1], c, -ms_lo));
        sacc[nt][2] = fast_exp2(fmaf(sacc[nt][2], c, -ms_hi));
        sacc[nt][3] = fast_exp2(fmaf(sacc[nt][3], c, -ms_hi));
        l_lo += sacc[nt][0] + sacc[nt][1];
        l_hi += sacc[nt][2] + sacc[nt][3];
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < SROWS / 16; ++kk) {
        uint32_t pa[4];
        pa[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
        pa[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
        pa[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
        pa[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
        const int r = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int np = 0; np < D / 16; ++np) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(vbase + tile_off(r, 2 * np + (lane >> 4)), b0, b1, b2, b3);
            mma_bf16(o[2 * np], pa, b0, b1);
            mma_bf16(o[2 * np + 1], pa, b2, b3);
        }
    }
}

template <int D>
__global__ void __launch_bounds__(THREADS, 1)
attn_mma_kernel(const AttnParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                const int nstage)
{
    constexpr int STAGE_BYTES = 2 * SROWS * D * 2;         // K rows + V rows of half a tile
    constexpr int MERGE_WARP_FLOATS = (D / 8 * 4 + 4) * 32;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    unsigned char* stages = smem;
    float* merge = reinterpret_cast<float*>(stages + (size_t)nstage * STAGE_BYTES);       // [6][MERGE_WARP_FLOATS]
    uint64_t* bars = reinterpret_cast<uint64_t*>(merge + 6 * MERGE_WARP_FLOATS);          // full[nstage], empty[nstage]
    int* pre = reinterpret_cast<int*>(bars + 2 * nstage);
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) abort_flag = 0;
    const long long total = scan_ntiles(p.ntiles, p.batch, pre);
    const long long U = total * p.hkv;
    if (U == 0) return;
    const long long lo = cta_first_unit(blockIdx.x, U, p.n_cta);
    const long long hi = cta_first_unit(blockIdx.x + 1, U, p.n_cta);
    if (lo >= hi) return;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + nstage);
    if (threadIdx.x == 0) {
        for (int i = 0; i < nstage; ++i) {
            mbar_init(full0 + 8 * i, 1);
            mbar_init(empty0 + 8 * i, NW);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    volatile int* abortp = &abort_flag;

    if (warp == NW) {
        // ------------------------------------------------ producer warp: lane 0 feeds the ring; the
        // tile ids are fetched 32 at a time by the whole warp so that no global-load latency sits
        // between two TMA issues
        int s = 0;
        uint32_t it = 0;
        long long u = lo;
        int ok = 1;
        while (u < hi && ok) {
            const Segment sg = decode_segment(u, hi, pre, p.hkv, s);
            for (int jb = sg.j0; jb < sg.j1 && ok; jb += 32) {
                const int jn = sg.j1 - jb < 32 ? sg.j1 - jb : 32;
                const int my_tile = lane < jn ? p.tiles[(size_t)sg.s * p.ntile_max + jb + lane] : 0;
                for (int k = 0; k < jn && ok; ++k) {
                    const int tile = __shfl_sync(0xffffffffu, my_tile, k);
                    if (lane == 0) {
                        for (int half = 0; half < HALVES && ok; ++half, ++it) {
                            const int st = it % nstage;
                            const uint32_t ph = (it / nstage) & 1;
                            if (!mbar_wait(empty0 + 8 * st, ph ^ 1, abortp, p.status)) { ok = 0; break; }
                            const int row0 = tile * TILE + half * SROWS;
                            const uint32_t dst = smem_u32(stages + (size_t)st * STAGE_BYTES);
                            mbar_expect_tx(full0 + 8 * st, STAGE_BYTES);
#pragma unroll
                            for (int h = 0; h < D / 64; ++h) {
                                tma_load_4d(dst + h * (SROWS * 128), &tm_k, full0 + 8 * st, h * 64, row0, sg.g, sg.s);
                                tma_load_4d(dst + SROWS * D * 2 + h * (SROWS * 128), &tm_v, full0 + 8 * st, h * 64, row0, sg.g, sg.s);
                            }
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                }
            }
            u = sg.next_u;
        }
        if (!ok && lane == 0) {
            // give the copies already in flight a bounded chance to land before the CTA ends
            const uint32_t first = it > (uint32_t)nstage ? it - nstage : 0;
            for (uint32_t k = first; k < it; ++k) {
                const uint32_t bar = full0 + 8 * (k % nstage), ph = (k / nstage) & 1;
                for (uint32_t i = 0; i < (1u << 16) && !mbar_try(bar, ph); ++i) __nanosleep(64);
            }
        }
        return;
    }

    // ---------------------------------------------------- consumers
    const float c = p.scale_log2;
    const __nv_bfloat16* __restrict__ Qg = reinterpret_cast<const __nv_bfloat16*>(p.q);
    const int gq = lane >> 2, cq = lane & 3;
    int s = 0;
    uint32_t it = 0;
    long long u = lo;
    bool alive = true;
    while (u < hi) {
        const Segment sg = decode_segment(u, hi, pre, p.hkv, s);
        const int A = p.n_active[sg.s];
        const int M = A * p.group;
        const int nmb = (M + 15) >> 4;
        const int kvl = nmb == 1 ? 4 : (nmb == 2 ? 4 : (nmb <= 4 ? 2 : 1));
        const bool active = warp < nmb * kvl;
        const int mb = active ? warp % nmb : 0, kl = active ? warp / nmb : 0;
        const int row_lo = mb * 16 + gq, row_hi = row_lo + 8;
        const int b_lo = row_lo / p.group, b_hi = row_hi / p.group;

        uint32_t qf[D / 16][4];
        float o[D / 8][4];
        float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        if (active) {
            // A fragments of the query block: row m = branch * group + head-in-group
            const size_t q_lo = (((size_t)sg.s * p.max_active + b_lo) * p.hq + (size_t)sg.g * p.group + (row_lo - b_lo * p.group)) * D;
            const size_t q_hi = (((size_t)sg.s * p.max_active + b_hi) * p.hq + (size_t)sg.g * p.group + (row_hi - b_hi * p.group)) * D;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const int d0 = ks * 16 + 2 * cq;
                qf[ks][0] = row_lo < M ? *reinterpret_cast<const uint32_t*>(Qg + q_lo + d0) : 0u;
                qf[ks][1] = row_hi < M ? *reinterpret_cast<const uint32_t*>(Qg + q_hi + d0) : 0u;
                qf[ks][2] = row_lo < M ? *reinterpret_cast<const uint32_t*>(Qg + q_lo + d0 + 8) : 0u;
                qf[ks][3] = row_hi < M ? *reinterpret_cast<const uint32_t*>(Qg + q_hi + d0 + 8) : 0u;
            }
        } else {
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) qf[ks][0] = qf[ks][1] = qf[ks][2] = qf[ks][3] = 0u;
        }
        const uint64_t* mrow_lo = p.mask + ((size_t)sg.s * p.max_active + (row_lo < M ? b_lo : 0)) * p.W;
        const uint64_t* mrow_hi = p.mask + ((size_t)sg.s * p.max_active + (row_hi < M ? b_hi : 0)) * p.W;

        for (int jb = sg.j0; jb < sg.j1; jb += 32) {
          const int jn = sg.j1 - jb < 32 ? sg.j1 - jb : 32;
          const int my_tile = lane < jn ? p.tiles[(size_t)sg.s * p.ntile_max + jb + lane] : 0;
          for (int q = HALVES * jb; q < HALVES * (jb + jn); ++q, ++it) {
            const int tile = __shfl_sync(0xffffffffu, my_tile, q / HALVES - jb);
            const int st = it % nstage;
            const uint32_t ph = (it / nstage) & 1;
            const bool mine = active && ((q - HALVES * sg.j0) % kvl) == kl;     // this KV lane's stage
            if (alive) {
                // every warp follows the ring (its arrival is counted), only the owners read the stage
                if (mine) {
                    if (!mbar_wait(full0 + 8 * st, ph, abortp, p.status)) alive = false;
                } else {
                    int ok = 1;
                    if (lane == 0) ok = mbar_wait(full0 + 8 * st, ph, abortp, p.status);
                    if (!__shfl_sync(0xffffffffu, ok, 0)) alive = false;
                }
            }
            if (alive && mine) {
                const int r0 = tile * TILE;
                const int sh = (q % HALVES) * SROWS;
                const bool masked = r0 + sh + SROWS > p.P;
                const uint64_t stage_bits = SROWS == 64 ? ~0ull : ((1ull << (SROWS & 63)) - 1ull);
                uint64_t mk_lo = ~0ull, mk_hi = ~0ull, zero_rows = 0ull;
                if (masked) {
                    mk_lo = row_lo < M ? (tile_rowmask(mrow_lo, p.W, p.P, tile) >> sh) & stage_bits : 0ull;
                    mk_hi = row_hi < M ? (tile_rowmask(mrow_hi, p.W, p.P, tile) >> sh) & stage_bits : 0ull;
                    uint64_t um = 0ull;                      // rows of the tile visible to any branch
                    for (int b = lane; b < A; b += 32)
                        um |= tile_rowmask(p.mask + ((size_t)sg.s * p.max_active + b) * p.W, p.W, p.P, tile);
                    const uint32_t ul = __reduce_or_sync(0xffffffffu, (uint32_t)um);
                    const uint32_t uh = __reduce_or_sync(0xffffffffu, (uint32_t)(um >> 32));
                    zero_rows = (~((((uint64_t)uh << 32) | ul) >> sh)) & stage_bits;
                }
                unsigned char* stg = stages + (size_t)st * STAGE_BYTES;
                const uint32_t kb = smem_u32(stg), vb = kb + SROWS * D * 2;
                process_stage<D>(kb, vb, stg + SROWS * D * 2, qf, o, m_lo, m_hi, l_lo, l_hi, masked, mk_lo, mk_hi, zero_rows,
                                 c, lane);
                if (masked) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * st);
          }
        }

        // ---- end of segment: merge the KV lanes, write the partial (m, l, O)
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
        if (active && kl > 0) {
            float* mbuf = merge + (size_t)((kl - 1) * nmb + mb) * MERGE_WARP_FLOATS;
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e) mbuf[(i * 4 + e) * 32 + lane] = o[i][e];
            mbuf[(D / 2 + 0) * 32 + lane] = m_lo;
            mbuf[(D / 2 + 1) * 32 + lane] = m_hi;
            mbuf[(D / 2 + 2) * 32 + lane] = l_lo;
            mbuf[(D / 2 + 3) * 32 + lane] = l_hi;
        }
        consumer_bar();
        if (active && kl == 0) {
            float mt_lo = m_lo, mt_hi = m_hi;
            for (int k2 = 1; k2 < kvl; ++k2) {
                const float* mbuf = merge + (size_t)((k2 - 1) * nmb + mb) * MERGE_WARP_FLOATS;
                mt_lo = fmaxf(mt_lo, mbuf[(D / 2 + 0) * 32 + lane]);
                mt_hi = fmaxf(mt_hi, mbuf[(D / 2 + 1) * 32 + lane]);
            }
            const float ms_lo = mt_lo == -INFINITY ? 0.f : mt_lo * c, ms_hi = mt_hi == -INFINITY ? 0.f : mt_hi * c;
            float w_lo = fast_exp2(m_lo * c - ms_lo), w_hi = fast_exp2(m_hi * c - ms_hi);
            l_lo *= w_lo;
            l_hi *= w_hi;
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                o[i][0] *= w_lo;
                o[i][1] *= w_lo;
                o[i][2] *= w_hi;
                o[i][3] *= w_hi;
            }
            for (int k2 = 1; k2 < kvl; ++k2) {
                const float* mbuf = merge + (size_t)((k2 - 1) * nmb + mb) * MERGE_WARP_FLOATS;
                w_lo = fast_exp2(mbuf[(D / 2 + 0) * 32 + lane] * c - ms_lo);
                w_hi = fast_exp2(mbuf[(D / 2 + 1) * 32 + lane] * c - ms_hi);
                l_lo = fmaf(mbuf[(D / 2 + 2) * 32 + lane], w_lo, l_lo);
                l_hi = fmaf(mbuf[(D / 2 + 3) * 32 + lane], w_hi, l_hi);
#pragma unroll
                for (int i = 0; i < D / 8; ++i) {
                    o[i][0] = fmaf(mbuf[(i * 4 + 0) * 32 + lane], w_lo, o[i][0]);
                    o[i][1] = fmaf(mbuf[(i * 4 + 1) * 32 + lane], w_lo, o[i][1]);
                    o[i][2] = fmaf(mbuf[(i * 4 + 2) * 32 + lane], w_hi, o[i][2]);
                    o[i][3] = fmaf(mbuf[(i * 4 + 3) * 32 + lane], w_hi, o[i][3]);
                }
            }
            const int slot = blockIdx.x + sg.s * p.hkv + sg.g;
            float* wo = p.ws_o + (size_t)slot * p.mmax * D;
            float* wml = p.ws_ml + (size_t)slot * p.mmax * 2;
            if (alive) {
                if (row_lo < M) {
#pragma unroll
                    for (int i = 0; i < D / 8; ++i)
                        *reinterpret_cast<float2*>(wo + (size_t)row_lo * D + i * 8 + 2 * cq) = make_float2(o[i][0], o[i][1]);
                    if (cq == 0) *reinterpret_cast<float2*>(wml + 2 * row_lo) = make_float2(mt_lo * c, l_lo);
                }
                if (row_hi < M) {
#pragma unroll
                    for (int i = 0; i < D / 8; ++i)
                        *reinterpret_cast<float2*>(wo + (size_t)row_hi * D + i * 8 + 2 * cq) = make_float2(o[i][2], o[i][3]);
                    if (cq == 0) *reinterpret_cast<float2*>(wml + 2 * row_hi) = make_float2(mt_hi * c, l_hi);
                }
            }
        }
        consumer_bar();            // the merge buffer is free again
        u = sg.next_u;
    }
}

// ---------------------------------------------------------------- host side
PFN_cuTensorMapEncodeTiled get_encode()
{
    static PFN_cuTensorMapEncodeTiled fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (PFN_cuTensorMapEncodeTiled)f;
    });
    return fn;
}

struct MapKey {
    const void* base;
    int64_t ss, sh, sr;
    int32_t batch, hkv, rows, d, box_rows, dev;
    bool operator==(const MapKey& o) const
    {
        return dev == o.dev && base == o.base && ss == o.ss && sh == o.sh && sr == o.sr && batch == o.batch && hkv == o.hkv && rows == o.rows && d == o.d && box_rows == o.box_rows;
    }
};
struct MapCache {
    std::mutex mu;
    std::vector<std::pair<MapKey, CUtensorMap>> items;
};
MapCache g_maps;

int get_map(const void* base, const AttnParams& p, int d, int box_rows, CUtensorMap* out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FDC_ERR_CUDA;
    MapKey key{base, p.stride_scene, p.stride_head, p.stride_row, p.batch, p.hkv, p.rows, d, box_rows, dev};
    std::lock_guard<std::mutex> lk(g_maps.mu);
    for (auto& it : g_maps.items)
        if (it.first == key) {
            *out = it.second;
            return FDC_OK;
        }
    PFN_cuTensorMapEncodeTiled enc = get_encode();
    if (!enc) return FDC_ERR_CUDA;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)p.rows, (cuuint64_t)p.hkv, (cuuint64_t)p.batch};
    // a dimension of extent 1 still needs a legal (multiple of 16 bytes, non-zero) stride
    auto str = [](int64_t s, int64_t fallback) { return (cuuint64_t)((s > 0 ? s : fallback) * 2); };
    cuuint64_t strides[3] = {str(p.stride_row, d), str(p.stride_head, (int64_t)d * p.rows), str(p.stride_scene, (int64_t)d * p.rows * p.hkv)};
    cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    alignas(64) CUtensorMap tm;
    CUresult r = enc(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return FDC_ERR_SHAPE;
    if (g_maps.items.size() >= 4096) g_maps.items.clear();
    g_maps.items.emplace_back(key, tm);
    *out = tm;
    return FDC_OK;
}

template <int D>
int launch_t(const AttnParams& p, cudaStream_t st)
{
    constexpr int STAGE_BYTES = 2 * SROWS * D * 2;
    constexpr int MERGE_BYTES = 6 * (D / 8 * 4 + 4) * 32 * 4;
    const size_t fixed = 1024 + MERGE_BYTES + 2 * 16 * 8 + sizeof(int) * (p.batch + 1) + 64;
    int nstage = (int)((227 * 1024 - 256 - fixed) / STAGE_BYTES);   // 256: static shared + slack
    if (nstage > 16) nstage = 16;
    if (nstage < 2) return FDC_ERR_SHAPE;
    const size_t smem = fixed + (size_t)nstage * STAGE_BYTES;
    static size_t attr_smem[kMaxDevices] = {};
    int rc = raise_dynamic_smem(reinterpret_cast<const void*>(attn_mma_kernel<D>), smem, attr_smem);
    if (rc) return rc;
    alignas(64) CUtensorMap tk, tv;
    rc = get_map(p.k, p, D, SROWS, &tk);
    if (rc) return rc;
    rc = get_map(p.v, p, D, SROWS, &tv);
    if (rc) return rc;
    attn_mma_kernel<D><<<p.n_cta, THREADS, smem, st>>>(p, tk, tv, nstage);
    note_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FDC_OK : set_cuda_error(e);
}

}  // namespace

namespace fdc {

int get_kv_tensor_map(const void* base, const AttnParams& p, int head_dim, int box_rows, void* out_map)
{
    return get_map(base, p, head_dim, box_rows, reinterpret_cast<CUtensorMap*>(out_map));
}

// bf16 only.  Returns FDC_ERR_SHAPE when the tensor map cannot describe the cache (the caller
// then uses the CUDA-core kernel).
int launch_attn_mma(const AttnParams& p, int head_dim, cudaStream_t st)
{
    return head_dim == 64 ? launch_t<64>(p, st) : launch_t<128>(p, st);
}

}  // namespace fdc
