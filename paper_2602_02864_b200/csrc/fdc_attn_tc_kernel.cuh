// Split-KV pass for bf16 caches (head_dim 128) on the 5th-generation tensor cores (tcgen05 + TMEM).
// This file is the whole kernel and its launcher; it is compiled twice, by the two translation
// units that include it with FDC_TC_NGRP = 1 and 2 (the number of groups the softmax warps work
// in, see softmax_segment), so that each build holds only its own inner loop and gets its own
// register allocation.
//
// Sec. 3.3: the queries of all parallel fields of a scene, times the GQA heads of a KV head,
// share ONE read of the KV rows.  The kernel is written in the transposed form, with the KV
// rows on the M side of the MMAs and the (few) query rows on the N side, so that the tensor
// work scales with the real number of queries and every TMEM lane / softmax thread owns a
// real KV row:
//     S^T = K Q^T      M = 128 KV rows (one "round" = two 64-row tiles of the visited-tile
//                      list), N = NP query rows (32/64/128), K = head_dim;  A = the K tiles
//                      as TMA left them in shared memory, B = Q^T staged once per segment
//     O^T += V^T P^T   M = head_dim, N = NP, K = 128 KV rows;  A = the V tiles (M-major), B =
//                      P^T written by the softmax threads (N-major), accumulator in TMEM
//     l   += P 1       M = 128 query columns, N = 16 columns of ones, K = 128 KV rows: the
//                      softmax denominators, from the same bf16 P^T as the line above
// One persistent CTA per SM, 20 warps:
//   warp 16      TMA producer of both rings (K stages and V stages: 128 rows, 128B swizzle, L2
//                evict-first); polls both rings' free barriers, never blocks on one of them
//   warp 17      issues S^T = K Q^T (one elected thread); allocates / frees TMEM.  S^T has four
//                buffers in TMEM (two for 128 query rows), so K Q^T runs ahead of the softmax
//   warp 18      with fdc_set_fused_append, first writes the pass's new K/V rows that fall into
//                this CTA's tiles; then issues the column-sum multiplications (one elected thread)
//   warp 19      issues O^T += V^T P^T (one elected thread)
//   warps 0-15   softmax.  Thread = one KV row of the round (TMEM lane) x a quarter (one group) or
//                a half (two groups) of the query columns.  Eq. 1 is applied by select from the
//                branches' row bitmaps; prefix tiles skip it.  Beyond the prefix the same threads
//                clear the V rows that no branch may see (they can hold anything, NaN included,
//                and 0 * NaN must not reach the accumulator) before they hand P^T over.
// The softmax reference of a query column is set in the first round of a segment: inside the
// prefix from the score against the round's first row (visible to everybody), else from the
// column maximum (a column that sees no row yet borrows the round's highest maximum).  A score
// more than 2^16 above its reference leaves a note that all warps act on two or three rounds
// later (no barrier in the common path); a rise of more than 2^100 within those rounds is
// flagged.  Sums and accumulator use the same reference and the same rounded P^T, so the result
// is exact up to the rounding of P^T.
#if !defined(FDC_TC_NGRP) || !defined(FDC_TC_NPMAX)
#error "include from a translation unit that defines FDC_TC_NGRP (1 or 2), FDC_TC_NPMAX (32, 64 or 128), FDC_TC_KERNEL and FDC_TC_LAUNCH"
#endif
#include <cudaTypedefs.h>

#include <climits>

#include "fdc_attn_common.cuh"

using namespace fdc;

namespace {

constexpr int D = 128;                       // head_dim handled by this kernel
constexpr int TILE = FDC_TILE_ROWS;          // rows per entry of the visited-tile list
constexpr int RROWS = 2 * TILE;              // KV rows per round = M of S^T = K of O^T
constexpr int NGRP = FDC_TC_NGRP;            // groups the softmax warps work in (this build)
constexpr int NP_MAX = FDC_TC_NPMAX;         // padded query rows of the widest pair of the launches this build serves (32, 64 or 128)
static_assert((NP_MAX == 64) == (NGRP == 2), "two groups exactly for 33 to 64 query rows");
constexpr int NSOFT = 16;                    // softmax warps: 4 row quadrants x 4 column parts
constexpr int NPART = NSOFT / 4;             // column parts
constexpr int W_PROD = NSOFT, W_QK = NSOFT + 1, W_AUX = NSOFT + 2, W_PV = NSOFT + 3;
constexpr int THREADS = (NSOFT + 4) * 32;
constexpr uint32_t TMEM_COLS = 512;          // S^T buffers [0,256): 4 x 64 columns (2 x 128 for 128 query rows) | O^T [256,384) | sums [384,512)
constexpr uint32_t TM_O = 256;
constexpr uint32_t TM_L = 384;                // column sums [384, 400): accumulator of the multiplication by ones (lane n: query column n)
constexpr int PANEL = RROWS * 128;           // 128 rows x 128 bytes (64 bf16 columns)
constexpr int ONES_BYTES = 2048;             // B operand of the column-sum multiplication: 16 x 16 bf16 ones (the footprint of its layout)
constexpr int STAGE = (D / 64) * PANEL;      // one K (or V) stage: 128 rows x head_dim
constexpr int MAXST = 4;                     // stages per ring at most
constexpr float RAISE_LOG2 = 16.f;
// Event trace for development builds (-DFDC_TRACE=<CTA>): clock64 stamps of one CTA, per round and
// per segment, read back with fdc_tr_read.  Compiled out otherwise.
#ifdef FDC_TRACE
__device__ long long g_tr[64 * 16];
__device__ long long g_ts[80];
#define FDC_TRC ((int)blockIdx.x == FDC_TRACE)
#define FDC_TR(g, e) do { if (FDC_TRC && (g) < 64) g_tr[(g) * 16 + (e)] = clock64(); } while (0)
#define FDC_TS(e) do { if (FDC_TRC) g_ts[e] = clock64(); } while (0)
#define FDC_TSS(e) do { if (FDC_TRC && seg < 4) g_ts[16 + seg * 16 + (e)] = clock64(); } while (0)
#else
#define FDC_TR(g, e) do { } while (0)
#define FDC_TS(e) do { } while (0)
#define FDC_TSS(e) do { } while (0)
#endif
constexpr float UNSET = 1.0e30f;             // -reference of a column that has seen nothing yet
#ifndef FDC_W_PREFIX
#define FDC_W_PREFIX 4
#endif
#ifndef FDC_W_MASKED
#define FDC_W_MASKED 6
#endif
#ifndef FDC_W_PAIR
#define FDC_W_PAIR 32
#endif
constexpr int W_PREFIX = FDC_W_PREFIX;       // cost of a tile inside the prefix (the unit of the weighted work split is a quarter of it)
constexpr int W_MASKED = FDC_W_MASKED;       // cost of a tile beyond the prefix (bitmap selects, V clean-up): measured about 1.5 prefix tiles
constexpr int W_PAIR = FDC_W_PAIR;           // cost of finishing a (scene, KV head) pair (drain, partial write, next queries)
constexpr int UW = 64;                       // words of a scene's union bitmap kept in shared memory (when W <= UW)
constexpr int MIN_TILES = 8;                 // tiles per CTA below which fewer CTAs are used (small problems)
constexpr int MIN_UNITS = MIN_TILES * W_PREFIX;   // the same as a weighted length
static_assert(MIN_UNITS >= 2 * FDC_W_MASKED, "every part of a pair must contain the start of at least one tile");
constexpr int MBUF = 512;                    // bitmap words of a scene kept in shared memory (max_active * W): one buffer; 2 * MBUF for 128 query rows
constexpr int MBUF_MAX = 1024;

// ---------------------------------------------------------------- tcgen05 wrappers
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor (128-byte swizzle, descriptor version 1): start address,
// leading-dimension byte offset, stride-dimension byte offset, all in units of 16 bytes.
// K-major operand: SBO = distance of 8-row groups.  MN-major operand: LBO = distance of
// 64-element groups along M/N, SBO = distance of 8-row groups along K.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulate, bf16 A and B, M x N; mn_major = 1 makes
// BOTH operands MN-major (contiguous along M resp. N), 0 makes both K-major.
__device__ __forceinline__ uint32_t instr_desc(int m, int n, uint32_t mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (mn_major << 15) | (mn_major << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}
// One MMA (cta_group::1, kind::f16).  The descriptors are given as (low, high) words: the address
// field sits in the low word, so stepping through an operand is 32-bit arithmetic for the issuing thread.
__device__ __forceinline__ void umma2(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                      uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\tmov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

#define FDC_R8(v, o) "=r"(v[o + 0]), "=r"(v[o + 1]), "=r"(v[o + 2]), "=r"(v[o + 3]), "=r"(v[o + 4]), "=r"(v[o + 5]), "=r"(v[o + 6]), "=r"(v[o + 7])
#define FDC_I8(v, o) "r"(v[o + 0]), "r"(v[o + 1]), "r"(v[o + 2]), "r"(v[o + 3]), "r"(v[o + 4]), "r"(v[o + 5]), "r"(v[o + 6]), "r"(v[o + 7])
// N consecutive fp32 columns of this thread's TMEM lane (N = 8, 16 or 32).
template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&v)[N])
{
    static_assert(N == 8 || N == 16 || N == 32, "column count");
    if constexpr (N == 32) {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,"
            "%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
            : FDC_R8(v, 0), FDC_R8(v, 8), FDC_R8(v, 16), FDC_R8(v, 24)
            : "r"(taddr)
            : "memory");
    } else if constexpr (N == 16) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                     : FDC_R8(v, 0), FDC_R8(v, 8)
                     : "r"(taddr)
                     : "memory");
    } else {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];" : FDC_R8(v, 0) : "r"(taddr) : "memory");
    }
}
template <int N>
__device__ __forceinline__ void tmem_st(uint32_t taddr, const uint32_t (&v)[N])
{
    static_assert(N == 8 || N == 16 || N == 32, "column count");
    if constexpr (N == 32) {
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,"
            "%24,%25,%26,%27,%28,%29,%30,%31};"
            ::FDC_I8(v, 0), FDC_I8(v, 8), FDC_I8(v, 16), FDC_I8(v, 24), "r"(taddr)
            : "memory");
    } else if constexpr (N == 16) {
        asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
                     ::FDC_I8(v, 0), FDC_I8(v, 8), "r"(taddr)
                     : "memory");
    } else {
        asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};" ::FDC_I8(v, 0), "r"(taddr) : "memory");
    }
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Barrier of the softmax warps (a named barrier).  Every call site is reached by all sixteen warps
// the same number of times whatever happens: a warp whose bounded wait ran out goes on without
// waiting but still takes every one of these.
__device__ __forceinline__ void soft_sync() { asm volatile("bar.sync 1, %0;" ::"n"(NSOFT * 32) : "memory"); }

// The barrier inside the reference-raising path.  Whether a warp enters that path in a given round
// depends on data (a note left two or three rounds earlier), which a warp that no longer waits for anything
// may read too early; a named barrier there could then be waited at for ever.  So this one is an
// mbarrier with a bounded wait, one arrival per warp: the worst a straying warp can cause is that the
// others give up too (FDC_DEV_TIMEOUT).
static __device__ __noinline__ void raise_sync_slow(uint32_t bar, uint64_t tok, volatile int* abort_flag, int32_t* status)
{
    for (uint32_t i = 0; i < (1u << 18); ++i) {
        uint32_t ok;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar), "l"(tok) : "memory");
        if (ok) return;
        if ((i & 255u) == 255u && *abort_flag) return;
    }
    *abort_flag = 1;
    atomicOr(status, FDC_DEV_TIMEOUT);
}
__device__ __forceinline__ void raise_sync(uint32_t bar, volatile int* abort_flag, int32_t* status)
{
    __syncwarp();
    uint64_t tok = 0;
    if ((threadIdx.x & 31) == 0) asm volatile("mbarrier.arrive.shared::cta.b64 %0, [%1];" : "=l"(tok) : "r"(bar) : "memory");
    tok = __shfl_sync(0xffffffffu, tok, 0);
    raise_sync_slow(bar, tok, abort_flag, status);
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// Monotone map float -> int (for integer max reductions).
__device__ __forceinline__ int ord_of(float x)
{
    const int i = __float_as_int(x);
    return i ^ ((i >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float ord_to(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

// Small per-CTA state in static shared memory.  The raise path finds its barrier from the address of
// the abort flag (it is handed that address anyway).
struct __align__(8) CtaFlags {
    uint64_t raise_bar;              // mbarrier of the reference-raising path (raise_sync)
    int abort_flag;                  // a bounded wait ran out somewhere in the CTA
    int v_steps[4];
};
constexpr uint32_t RAISE_BAR_BEFORE_ABORT_FLAG = 8;
static_assert(offsetof(CtaFlags, abort_flag) - offsetof(CtaFlags, raise_bar) == RAISE_BAR_BEFORE_ABORT_FLAG, "layout");

// Everything a role needs to find its barriers and buffers.
struct Ctx {
    // mbarriers: one base address, fixed offsets (kept as functions so that a single register serves them all)
    uint32_t bar0;
    __device__ __forceinline__ uint32_t k_full() const { return bar0; }
    __device__ __forceinline__ uint32_t k_empty() const { return bar0 + 8 * MAXST; }
    __device__ __forceinline__ uint32_t v_full() const { return bar0 + 16 * MAXST; }
    __device__ __forceinline__ uint32_t v_empty() const { return bar0 + 24 * MAXST; }
    __device__ __forceinline__ uint32_t s_full() const { return bar0 + 32 * MAXST; }
    __device__ __forceinline__ uint32_t s_free() const { return bar0 + 32 * MAXST + 32; }
    __device__ __forceinline__ uint32_t p_full() const { return bar0 + 32 * MAXST + 64; }
    __device__ __forceinline__ uint32_t pv_done() const { return bar0 + 32 * MAXST + 80; }
    __device__ __forceinline__ uint32_t q_ready() const { return bar0 + 32 * MAXST + 96; }
    __device__ __forceinline__ uint32_t o_free() const { return bar0 + 32 * MAXST + 104; }
    __device__ __forceinline__ uint32_t app_done() const { return bar0 + 32 * MAXST + 112; }
    int ns, s_stride;                // S^T buffers in TMEM (4 of 64 columns up to 64 query rows, else 2 of 128) and their distance
    uint32_t tmem;
    unsigned char *kring, *vring, *qs, *ps, *ones;
    float *mneg, *alpha, *lred;      // [128] -reference per column, [128] rescale factors, [4][128] partial sums
    int *cmax, *flags;               // [128] column maxima (ordered ints), [4] flags of the raise path and the merge
    int* rflag;                      // [8] rflag[g & 7] == g: round g met a score far above its reference
    int *pre, *nact;                 // [batch + 1] tile prefix sums, [batch] active branches per scene
    uint64_t* smask;                 // [2][mbuf] the current segment's scene bitmaps (when mstaged)
    int mbuf;                        // words per buffer
    uint64_t* sunion;                // [2][UW] their OR over the scene's active branches (when mstaged and W <= UW)
    int mstaged;
    int n_cta;                       // CTAs that take part: at most the grid, at least MIN_UNITS tiles each
    int* prev;                       // [batch + 1] prefix sums over scenes (per KV head) of parts (tpart > 0) or weighted lengths; or nullptr
    int tpart;                       // > 0: every CTA owns one part (at most tpart tiles) of one pair
    int npre;                        // tiles wholly inside the prefix
    long long vtot;                  // total weighted length
    volatile int* abortp;
    volatile int* v_steps;           // [2][2] per P^T buffer and tile of the round: the 16-row steps to multiply (bit k: rows 16k..)
    int nk, nv, q_panel, p_buf, npb; // ring depths, bytes per 64-column panel of Q^T, bytes per P^T buffer, P^T buffers (1 or 2)
};

// Row bitmap (Eq. 1) of branch b of the segment's scene.  While the K/V stream saturates the
// memory system a global read costs microseconds, so the softmax warps copy the scene's bitmaps
// to shared memory at the start of a segment whenever they fit.
__device__ __forceinline__ const uint64_t* mask_row(const AttnParams& p, const Ctx& cx, uint32_t seg, int s, int b)
{
    return cx.mstaged ? cx.smask + (seg & 1) * cx.mbuf + (size_t)b * p.W : p.mask + ((size_t)s * p.max_active + b) * p.W;
}
// 16-byte asynchronous copy global -> shared (zero fill when !valid); completes with cp_async_wait_all.
__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async8(void* dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// ---- weighted work split ---------------------------------------------------------------------
// CTAs get equal shares of a WEIGHTED length, not of the tile count: a tile beyond the prefix
// costs W_MASKED / W_PREFIX prefix tiles and the end of every pair costs W_PAIR / W_PREFIX.  Tile j of a pair starts at
// weighted offset vt(j); a pair of nt tiles is vt(nt) + W_PAIR long.  A CTA owns the tiles whose
// start falls into its share, so shares always cut the unit sequence into consecutive runs.
__device__ __forceinline__ int vt_of(const Ctx& cx, int nt, int j)
{
    const int np = cx.npre < nt ? cx.npre : nt;
    return j <= np ? j * W_PREFIX : np * W_PREFIX + (j - np) * W_MASKED;
}
// First tile of a pair of nt tiles whose weighted start is >= r (nt if there is none).
__device__ __forceinline__ int tile_of_vt(const Ctx& cx, int nt, int r)
{
    const int np = cx.npre < nt ? cx.npre : nt;
    const int j = r <= np * W_PREFIX ? (r + W_PREFIX - 1) / W_PREFIX : np + (r - np * W_PREFIX + W_MASKED - 1) / W_MASKED;
    return j > nt ? nt : j;
}
// First unit whose weighted start is >= x.
__device__ __forceinline__ long long unit_of_virt(const AttnParams& p, const Ctx& cx, long long x)
{
    if (x >= cx.vtot) return (long long)cx.pre[p.batch] * p.hkv;
    int lo = 0, hi = p.batch;                      // largest s with prev[s] * hkv <= x
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long long)cx.prev[mid] * p.hkv <= x) lo = mid;
        else hi = mid;
    }
    int s = lo;
    while (cx.prev[s + 1] == cx.prev[s]) ++s;     // scenes without tiles have no length
    const int V = cx.prev[s + 1] - cx.prev[s], nt = cx.pre[s + 1] - cx.pre[s];
    const long long y = x - (long long)cx.prev[s] * p.hkv;
    const int g = (int)(y / V), r = (int)(y - (long long)g * V);
    return (long long)cx.pre[s] * p.hkv + (long long)g * nt + tile_of_vt(cx, nt, r);
}
// CTAs that hold the first and the last tile of pair (s, g).
__device__ __forceinline__ void pair_ctas(const AttnParams& p, const Ctx& cx, int s, int g, int& c_first, int& c_last)
{
    const int nt = cx.pre[s + 1] - cx.pre[s];
    if (cx.tpart) {                                // one part per CTA: the pair's parts are consecutive CTAs
        const int k = cx.prev[s + 1] - cx.prev[s];
        c_first = cx.prev[s] * p.hkv + g * k;
        c_last = c_first + k - 1;
    } else if (!cx.prev) {
        const long long u0 = (long long)cx.pre[s] * p.hkv + (long long)g * nt, U = (long long)cx.pre[p.batch] * p.hkv;
        c_first = unit_cta(u0, U, cx.n_cta);
        c_last = unit_cta(u0 + nt - 1, U, cx.n_cta);
    } else {
        const long long v0 = (long long)cx.prev[s] * p.hkv + (long long)g * (cx.prev[s + 1] - cx.prev[s]);
        c_first = (int)((v0 * cx.n_cta) / cx.vtot);
        c_last = (int)(((v0 + vt_of(cx, nt, nt - 1)) * cx.n_cta) / cx.vtot);
    }
}

// Position of one ring's producer in the CTA's unit sequence.
struct Cursor {
    long long u;                 // first unit of the current segment
    Segment sg;
    int s, jb, jn, k, my_tile;   // scene hint; batch of up to 32 tile ids (one per lane) and the position inside it
    uint32_t g;                  // round
    int st;                      // ring stage of round g
    uint32_t ph;                 // ring phase of round g
    int live;
};
__device__ __forceinline__ void cursor_batch(Cursor& c, const AttnParams& p, int lane)
{
    c.jn = c.sg.j1 - c.jb < 32 ? c.sg.j1 - c.jb : 32;
    // entry j of a tile list is tile j for every whole tile of the prefix: no need to read those
    const int j = c.jb + lane;
    c.my_tile = lane < c.jn ? (j < p.P / TILE ? j : p.tiles[(size_t)c.sg.s * p.ntile_max + j]) : 0;
    c.k = 0;
}
__device__ __forceinline__ void cursor_open(Cursor& c, const AttnParams& p, const Ctx& cx, long long hi, int lane)
{
    c.live = c.u < hi;
    if (!c.live) return;
    c.sg = decode_segment(c.u, hi, cx.pre, p.hkv, c.s);
    c.jb = c.sg.j0;
    cursor_batch(c, p, lane);
}
__device__ __forceinline__ void cursor_next(Cursor& c, const AttnParams& p, const Ctx& cx, long long hi, int nst, int lane)
{
    c.k += 2;
    ++c.g;
    if (++c.st == nst) {
        c.st = 0;
        c.ph ^= 1;
    }
    if (c.k < c.jn) return;
    c.jb += 32;
    if (c.jb < c.sg.j1) {
        cursor_batch(c, p, lane);
    } else {
        c.u = c.sg.next_u;
        cursor_open(c, p, cx, hi, lane);
    }
}
// Does the round at the cursor reach beyond the prefix?  (whole warp; tile ids ascend)
__device__ __forceinline__ bool cursor_beyond_prefix(const Cursor& c, int P)
{
    const int nt = c.jn - c.k < 2 ? 1 : 2;
    return __shfl_sync(0xffffffffu, c.my_tile, (c.k + nt - 1) & 31) * TILE + TILE > P;
}
// The round at the cursor: two tiles (rows 0-63 and 64-127 of both 64-column panels) into one stage.
__device__ __forceinline__ void cursor_issue(const Cursor& c, const CUtensorMap* tm, unsigned char* ring, uint32_t full, uint64_t pol, int lane)
{
    const int nt = c.jn - c.k < 2 ? 1 : 2;
    const int t0 = __shfl_sync(0xffffffffu, c.my_tile, c.k);
    const int t1 = __shfl_sync(0xffffffffu, c.my_tile, (c.k + 1) & 31);
    if (lane == 0) {
        const uint32_t dst = smem_u32(ring + (size_t)c.st * STAGE);
        mbar_expect_tx(full + 8 * c.st, nt * (STAGE / 2));
#pragma unroll
        for (int h = 0; h < D / 64; ++h) {
            tma_load_4d_hint(dst + h * PANEL, tm, full + 8 * c.st, h * 64, t0 * TILE, c.sg.g, c.sg.s, pol);
            if (nt == 2) tma_load_4d_hint(dst + h * PANEL + TILE * 128, tm, full + 8 * c.st, h * 64, t1 * TILE, c.sg.g, c.sg.s, pol);
        }
    }
}

// One TMA producer warp for both rings: whichever of the next K stage and the next V stage is
// free gets its round's tiles; the warp never blocks on one ring while the other could be fed.
__device__ __forceinline__ void producer_loop(const AttnParams& p, const Ctx& cx, const CUtensorMap* tm_k, const CUtensorMap* tm_v,
                                              long long lo, long long hi, int lane)
{
    const uint64_t pol = l2_evict_first_policy();     // every KV row is read once per call
    Cursor ck, cv;
    ck.u = lo;
    ck.s = 0;
    ck.g = 0;
    ck.st = 0;
    ck.ph = 0;
    cursor_open(ck, p, cx, hi, lane);
    cv = ck;
    int ok = 1;
    uint32_t idle = 0;
    int app_ok = p.app_row == nullptr;               // rows appended by this kernel are in place (tiles beyond the prefix may be loaded)
    int waited = !p.early;                           // the kernel ahead in the stream has completed (griddepcontrol.wait was taken)
    int q_hold = p.early;                            // after the wait, the first pair's queries go ahead of further K/V requests
    while ((ck.live || cv.live) && ok) {
        if (!app_ok && waited) {
            const int done = lane == 0 ? (int)mbar_try(cx.app_done(), 0) : 0;
            app_ok = __shfl_sync(0xffffffffu, done, 0);
        }
        // Rows beyond the prefix may have been written by the kernel ahead (fdc_kv_append) or are written
        // by this one (fused append): their tiles wait for both.  Prefix rows never change during decode.
        if (q_hold && waited) {
            // The queries are requested right after the wait; whatever this SM requests before them
            // arrives before them.  The stages requested ahead of the wait keep the first rounds fed.
            const int done = lane == 0 ? (int)mbar_try(cx.q_ready(), 0) : 0;
            q_hold = !__shfl_sync(0xffffffffu, done, 0);
        }
        const bool hold_all = q_hold && waited;
        const bool hold_k = hold_all || (!(app_ok && waited) && ck.live && cursor_beyond_prefix(ck, p.P));
        const bool hold_v = hold_all || (!(app_ok && waited) && cv.live && cursor_beyond_prefix(cv, p.P));
        int rk = 0, rv = 0;
        if (lane == 0) {
            rk = ck.live && !hold_k && mbar_try(cx.k_empty() + 8 * ck.st, ck.ph ^ 1);
            rv = cv.live && !hold_v && mbar_try(cx.v_empty() + 8 * cv.st, cv.ph ^ 1);
        }
        rk = __shfl_sync(0xffffffffu, rk, 0);
        rv = __shfl_sync(0xffffffffu, rv, 0);
        if (rk) {
            if (lane == 0) FDC_TR(ck.g, 12);
            cursor_issue(ck, tm_k, cx.kring, cx.k_full(), pol, lane);
            cursor_next(ck, p, cx, hi, cx.nk, lane);
        }
        if (rv) {
            if (lane == 0) FDC_TR(cv.g, 13);
            cursor_issue(cv, tm_v, cx.vring, cx.v_full(), pol, lane);
            cursor_next(cv, p, cx, hi, cx.nv, lane);
        }
        if (rk | rv) {
            idle = 0;
        } else if (!waited) {
            // nothing more can be requested ahead of the kernel before this one: wait for it to complete
            asm volatile("griddepcontrol.wait;" ::: "memory");
            waited = 1;
        } else if (((++idle) & 63u) == 0u) {
            // bounded: no stage became free for a long time, or another role gave up
            if (idle >= SPIN_LIMIT) {
                if (lane == 0) {
                    *cx.abortp = 1;
                    atomicOr(p.status, FDC_DEV_TIMEOUT);
                }
                ok = 0;
            } else if (*cx.abortp) {
                ok = 0;
            } else {
                __nanosleep(32);
            }
        }
    }
    if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");     // (a run wholly inside the prefix that fitted the rings)
    if (!ok && lane == 0) {
        // give the copies already in flight a bounded chance to land before the CTA ends
        for (int r = 0; r < 2; ++r) {
            const uint32_t g = r ? cv.g : ck.g, nst = r ? cx.nv : cx.nk, full = r ? cx.v_full() : cx.k_full();
            const uint32_t first = g > nst ? g - nst : 0;
            for (uint32_t k = first; k < g; ++k) {
                const uint32_t bar = full + 8 * (k % nst), ph = (k / nst) & 1;
                for (uint32_t i = 0; i < (1u << 16) && !mbar_try(bar, ph); ++i) __nanosleep(64);
            }
        }
    }
}

// One elected thread: S^T[g mod ns] = K(stage) Q^T for every round g.  A score buffer is free again
// once the softmax threads have read round g - ns (s_free); with four buffers K Q^T runs well ahead of
// the softmax, so a K stage is released soon after it landed and the K ring stays in flight.
__device__ __forceinline__ void qk_loop(const AttnParams& p, const Ctx& cx, long long lo, long long hi, int lane)
{
    const uint64_t q_desc = smem_desc(smem_u32(cx.qs), 16, 1024);
    const uint64_t k_desc0 = smem_desc(smem_u32(cx.kring), 16, 1024);
    const uint32_t q_lo = (uint32_t)q_desc, q_hi = (uint32_t)(q_desc >> 32), k_lo0 = (uint32_t)k_desc0, k_hi = (uint32_t)(k_desc0 >> 32);
    const uint32_t qp16 = (uint32_t)(cx.q_panel >> 4);
    int s = 0;
    uint32_t g = 0, seg = 0;
    int st = 0;
    uint32_t kph = 0;                               // ring position and phase of the K stage of round g
    long long u = lo;
    int ok = 1;
    while (u < hi && ok) {
        const Segment sg = decode_segment(u, hi, cx.pre, p.hkv, s);
        const int nr = (sg.j1 - sg.j0 + 1) >> 1;
        if (lane == 0) {
            const int M = cx.nact[sg.s] * p.group;
            const int NP = (NP_MAX == 32 || M <= 32) ? 32 : ((NP_MAX == 64 || M <= 64) ? 64 : 128);
            const uint32_t idesc_qk = instr_desc(RROWS, NP, 0);
            bool good = mbar_wait(cx.q_ready(), seg & 1, cx.abortp, p.status);
            for (int t = 0; t < nr && good; ++t, ++g) {
                good = mbar_wait(cx.k_full() + 8 * st, kph, cx.abortp, p.status);
                FDC_TR(g, 6);
                const uint32_t sb = g & (cx.ns - 1);                  // score buffer of the round
                if (good && g >= (uint32_t)cx.ns) good = mbar_wait(cx.s_free() + 8 * sb, ((g / cx.ns) - 1) & 1, cx.abortp, p.status);
                if (!good) break;
                FDC_TR(g, 7);
                tc_fence_after();
                const uint32_t kd = k_lo0 + (uint32_t)((st * STAGE) >> 4);
                const uint32_t d = cx.tmem + sb * cx.s_stride;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    umma2(d, kd + (uint32_t)(((ks >> 2) * PANEL + (ks & 3) * 32) >> 4), k_hi, q_lo + (ks >> 2) * qp16 + (uint32_t)(((ks & 3) * 32) >> 4), q_hi,
                          idesc_qk, ks > 0);
                umma_commit(cx.k_empty() + 8 * st);
                umma_commit(cx.s_full() + 8 * sb);
                FDC_TR(g, 8);
                if (++st == cx.nk) {
                    st = 0;
                    kph ^= 1;
                }
            }
            ok = good;
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        g = __shfl_sync(0xffffffffu, g, 0);
        st = __shfl_sync(0xffffffffu, st, 0);
        kph = __shfl_sync(0xffffffffu, kph, 0);
        ++seg;
        u = sg.next_u;
    }
}

// Fused append (one warp; out of line, all arguments by value).  The new K/V vectors of this pass
// (Sec. 3.3: every emitted token's K/V is written once, at the row its slot reserves) whose rows
// lie in KV tiles that this CTA owns are written here, before the CTA loads those tiles: every
// tile of a (scene, KV head) pair belongs to exactly one CTA, so every vector is written exactly
// once and no CTA depends on another.  Lanes 0-15 copy the 16 chunks of a K row, lanes 16-31
// those of the V row.  Rows outside [P, rows) are skipped and flagged.  The writes are made
// visible to the TMA loads (asynchronous proxy) of this CTA before the caller signals them.
__device__ __noinline__ void append_rows(char* kc, char* vc, long long stride_scene_b, long long stride_head_b, long long stride_row_b,
                                         const int32_t* app_row, const char* app_k, const char* app_v, const int32_t* tiles,
                                         int ntile_max, int max_active, int hkv, int rows, int P, const int* pre, const int* nact,
                                         long long lo, long long hi, int32_t* status)
{
    const int lane = threadIdx.x & 31;
    const int chunk = (lane & 15) * 16;
    const char* src_base = lane < 16 ? app_k : app_v;
    char* dst_base = lane < 16 ? kc : vc;
    int s = 0;
    long long u = lo;
    while (u < hi) {
        const Segment sg = decode_segment(u, hi, pre, hkv, s);
        const int A = nact[sg.s];
        const int t_first = tiles[(size_t)sg.s * ntile_max + sg.j0], t_last = tiles[(size_t)sg.s * ntile_max + sg.j1 - 1];
        for (int b0 = 0; b0 < A; b0 += 32) {
            const int b = b0 + lane;
            const int r = b < A ? app_row[(size_t)sg.s * max_active + b] : P;
            const bool in_range = r >= P && r < rows;
            if (!in_range && sg.g == 0 && sg.j0 == 0) atomicOr(status, FDC_DEV_ROW_RANGE);      // once per scene
            const int t = r / TILE;
            unsigned m = __ballot_sync(0xffffffffu, b < A && in_range && t >= t_first && t <= t_last);
            while (m) {
                // up to four rows per turn, all loads before the first store
                uint4 val[4];
                long long dst[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    dst[i] = -1;
                    if (m) {
                        const int bi = __ffs(m) - 1;
                        m &= m - 1;
                        const int ri = __shfl_sync(0xffffffffu, r, bi);
                        const size_t slot = (size_t)sg.s * max_active + b0 + bi;
                        val[i] = *reinterpret_cast<const uint4*>(src_base + (slot * hkv + sg.g) * (D * 2) + chunk);
                        dst[i] = (long long)sg.s * stride_scene_b + (long long)sg.g * stride_head_b + (long long)ri * stride_row_b + chunk;
                    }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (dst[i] >= 0) *reinterpret_cast<uint4*>(dst_base + dst[i]) = val[i];
            }
        }
        u = sg.next_u;
    }
    __threadfence();
    asm volatile("fence.proxy.async;" ::: "memory");
    __syncwarp();
}

// Rows of a KV tile beyond the prefix that some branch of the scene may see (the OR of the
// branches' bitmaps; prefix rows of a tile that straddles the end of the prefix included).  `un` is
// that OR as the softmax warps prepared it per pair (the usual case), else nullptr and the bitmaps
// themselves are combined here (templates too long for the shared-memory copy).
__device__ __noinline__ uint64_t tile_seen_rows(const uint64_t* un, const uint64_t* mask0, int W, int P, int A, int tile)
{
    if (un) return tile_rowmask(un, W, P, tile);
    // (whole warp: the lanes share the branches and combine)
    const int lane = threadIdx.x & 31;
    uint64_t um = 0ull;
    for (int b = lane; b < A; b += 32) um |= tile_rowmask(mask0 + (size_t)b * W, W, P, tile);
    const uint32_t ul = __reduce_or_sync(0xffffffffu, (uint32_t)um);
    const uint32_t uh = __reduce_or_sync(0xffffffffu, (uint32_t)(um >> 32));
    return ((uint64_t)uh << 32) | ul;
}

// The auxiliary warp: with fdc_set_fused_append it writes the pass's new K/V rows that fall into
// this CTA's tiles, then lets the producer go on to the tiles beyond the prefix; after that one
// of its threads issues the column-sum multiplications.
__device__ __forceinline__ void aux_loop(const AttnParams& p, const Ctx& cx, long long lo, long long hi, int lane)
{
    if (p.app_row) {
        append_rows(const_cast<char*>(reinterpret_cast<const char*>(p.k)), const_cast<char*>(reinterpret_cast<const char*>(p.v)),
                    p.stride_scene * 2, p.stride_head * 2, p.stride_row * 2, p.app_row, reinterpret_cast<const char*>(p.app_k),
                    reinterpret_cast<const char*>(p.app_v), p.tiles, p.ntile_max, p.max_active, p.hkv, p.rows, p.P, cx.pre, cx.nact, lo, hi,
                    p.status);
        if (lane == 0) mbar_arrive(cx.app_done());
    }
    // The column sums of P^T (the softmax denominators), taken by the tensor core beside every
    // O^T += V^T P^T: P (128 query columns as rows, read from the same P^T buffer, which is laid out
    // the same way for either operand) times 16 columns of ones, so that TMEM lane n of the accumulator
    // holds sum_k P^T[k][n] of exactly the values that are multiplied with V.  For fewer than 128 query
    // rows the multiplication reads on past the P^T buffer (shared memory of this CTA all the same):
    // those rows of the result are never looked at, and a row depends on nothing but its own inputs.
    // Issued from this warp so that the thread that issues the V multiplications is not slowed down;
    // the same 16-row steps are left out, and both threads commit to the pv_done barrier.
    const uint64_t ones_desc = smem_desc(smem_u32(cx.ones), PANEL, 1024);
    const uint64_t p_desc0 = smem_desc(smem_u32(cx.ps), PANEL, 1024);
    const uint32_t ones_lo = (uint32_t)ones_desc, ones_hi = (uint32_t)(ones_desc >> 32), p_lo0 = (uint32_t)p_desc0, p_hi = (uint32_t)(p_desc0 >> 32);
    const uint32_t tm_l = cx.tmem + TM_L;
    int s = 0;
    uint32_t g = 0, seg = 0;
    long long u = lo;
    int ok = 1;
    while (u < hi && ok) {
        const Segment sg = decode_segment(u, hi, cx.pre, p.hkv, s);
        if (lane == 0) {
            const uint32_t idesc_sum = instr_desc(128, 16, 1);
            const int ntile = sg.j1 - sg.j0;
            bool good = true;
            for (int t = 0; 2 * t < ntile && good; ++t, ++g) {
                good = mbar_wait(cx.p_full() + 8 * (g & 1), (g >> 1) & 1, cx.abortp, p.status);
                if (good && t == 0 && seg > 0) good = mbar_wait(cx.o_free(), (seg - 1) & 1, cx.abortp, p.status);
                if (!good) break;
                const uint32_t steps = (uint32_t)cx.v_steps[(g & 1) * 2] | ((uint32_t)cx.v_steps[(g & 1) * 2 + 1] << 4);
                tc_fence_after();
                const uint32_t pd = p_lo0 + (uint32_t)((((g & 1) & (cx.npb - 1)) * cx.p_buf) >> 4);
                uint32_t acc = t > 0 ? 1u : 0u;
#pragma unroll 1
                for (int kk = 0; kk < 8; ++kk)
                    if ((steps >> kk) & 1u) {
                        umma2(tm_l, pd + kk * 128, p_hi, ones_lo, ones_hi, idesc_sum, acc);
                        acc = 1u;
                    }
                umma_commit(cx.pv_done() + 8 * (g & 1));
            }
            ok = good;
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        g = __shfl_sync(0xffffffffu, g, 0);
        ++seg;
        u = sg.next_u;
    }
}

// One elected thread: O^T += V^T(stage) P^T[g & 1] for every round g, once the stage has landed and
// the softmax warps have delivered P^T (and, beyond the prefix, cleared the stage's unseen rows).
// The multiplication runs in steps of 16 KV rows; the softmax warps say which steps hold a visible
// row (all of them inside the prefix), the others are left out.
__device__ __forceinline__ void pv_loop(const AttnParams& p, const Ctx& cx, long long lo, long long hi, int lane)
{
    const uint64_t v_desc0 = smem_desc(smem_u32(cx.vring), PANEL, 1024);
    const uint64_t p_desc0 = smem_desc(smem_u32(cx.ps), PANEL, 1024);
    const uint32_t v_lo0 = (uint32_t)v_desc0, v_hi = (uint32_t)(v_desc0 >> 32), p_lo0 = (uint32_t)p_desc0, p_hi = (uint32_t)(p_desc0 >> 32);
    const uint32_t tm_o = cx.tmem + TM_O;
    int s = 0;
    uint32_t g = 0, seg = 0;
    int st = 0;
    uint32_t vph = 0;
    long long u = lo;
    int ok = 1;
    while (u < hi && ok) {
        const Segment sg = decode_segment(u, hi, cx.pre, p.hkv, s);
        if (lane == 0) {
            const int M = cx.nact[sg.s] * p.group;
            const int NP = (NP_MAX == 32 || M <= 32) ? 32 : ((NP_MAX == 64 || M <= 64) ? 64 : 128);
            const uint32_t idesc_pv = instr_desc(D, NP, 1);
            const int ntile = sg.j1 - sg.j0;
            bool good = true;
            for (int t = 0; 2 * t < ntile && good; ++t, ++g) {
                good = mbar_wait(cx.v_full() + 8 * st, vph, cx.abortp, p.status);
                FDC_TR(g, 9);
                if (good) good = mbar_wait(cx.p_full() + 8 * (g & 1), (g >> 1) & 1, cx.abortp, p.status);
                if (good && t == 0 && seg > 0) good = mbar_wait(cx.o_free(), (seg - 1) & 1, cx.abortp, p.status);
                if (!good) break;
                FDC_TR(g, 10);
                const uint32_t steps = (uint32_t)cx.v_steps[(g & 1) * 2] | ((uint32_t)cx.v_steps[(g & 1) * 2 + 1] << 4);
                tc_fence_after();
                const uint32_t vd = v_lo0 + (uint32_t)((st * STAGE) >> 4);
                const uint32_t pd = p_lo0 + (uint32_t)((((g & 1) & (cx.npb - 1)) * cx.p_buf) >> 4);
                if (steps == 0xffu) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) umma2(tm_o, vd + kk * 128, v_hi, pd + kk * 128, p_hi, idesc_pv, (t > 0 || kk > 0) ? 1u : 0u);
                } else {
                    // a one-tile round has 64 KV rows; beyond the prefix, steps without a visible row are left out
                    // (rows that nobody may see can hold NaN, and 0 * NaN must not reach the accumulator)
                    uint32_t acc = t > 0 ? 1u : 0u;
#pragma unroll 1
                    for (int kk = 0; kk < 8; ++kk)
                        if ((steps >> kk) & 1u) {
                            umma2(tm_o, vd + kk * 128, v_hi, pd + kk * 128, p_hi, idesc_pv, acc);
                            acc = 1u;
                        }
                }
                umma_commit(cx.v_empty() + 8 * st);
                umma_commit(cx.pv_done() + 8 * (g & 1));
                FDC_TR(g, 11);
                if (++st == cx.nv) {
                    st = 0;
                    vph ^= 1;
                }
            }
            ok = good;
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        g = __shfl_sync(0xffffffffu, g, 0);
        st = __shfl_sync(0xffffffffu, st, 0);
        vph = __shfl_sync(0xffffffffu, vph, 0);
        ++seg;
        u = sg.next_u;
    }
}

// Visibility (Eq. 1) of one KV row for the nph (<= 32) query columns starting at col0: bit i <=>
// column col0 + i may see the row.  `row` (0..63) is the thread's row inside tile `tile`.  Columns
// b * G .. b * G + G - 1 belong to branch b; every thread reads the bitmap words of the two or three
// branches its columns belong to (the same words for the whole warp: one broadcast read each).
// When the prefix is a whole number of tiles a tile's 64 rows are one word of the bitmap; otherwise
// they straddle two (tile_rowmask).  Only tiles beyond the prefix come here.
__device__ __forceinline__ uint32_t row_visibility(const uint64_t* mask0, int W, int P, int tile, int row, int A, int G, int b_lo, int col0, int nph)
{
    uint32_t vis = 0u;
    const bool aligned = (P & (TILE - 1)) == 0;
    const int w = tile - P / TILE;
    int c = b_lo * G - col0;                       // first column of branch b relative to col0 (<= 0 for the first one)
#pragma unroll 1
    for (int b = b_lo; b < A && c < nph; ++b, c += G) {
        const uint64_t word = aligned ? (w < W ? mask0[(size_t)b * W + w] : 0ull) : tile_rowmask(mask0 + (size_t)b * W, W, P, tile);
        const int lo = c < 0 ? 0 : c, hi = c + G > nph ? nph : c + G;
        const uint32_t span = (hi - lo >= 32 ? 0xffffffffu : ((1u << (hi - lo)) - 1u)) << lo;
        if ((word >> row) & 1ull) vis |= span;
    }
    return vis;
}

// Asynchronous copies of the next segment's queries into Q^T and of its scene's bitmaps into
// the other bitmap buffer (softmax threads; completed with cp_async_wait_all in the prologue).
// (All arguments by value: a reference to the caller's context would force it into local memory.)
__device__ __noinline__ void prefetch_next_segment(const uint4* qg, const uint64_t* mask, int max_active, int W, int hq, int G, int hkv,
                                                   const int* pre, const int* nact, unsigned char* qs, int q_panel,
                                                   uint64_t* smask_dst, long long next_u, long long hi, int s_cur)
{
    const int tid = threadIdx.x;
    int s2 = s_cur;
    const Segment nx = decode_segment(next_u, hi, pre, hkv, s2);
    const int M2 = nact[nx.s] * G;
    const int NP2 = (NP_MAX == 32 || M2 <= 32) ? 32 : ((NP_MAX == 64 || M2 <= 64) ? 64 : 128);
    for (int idx = tid; idx < NP2 * (D / 8); idx += NSOFT * 32) {
        const int n = idx / (D / 8), ch = idx - n * (D / 8);
        const bool valid = n < M2;
        const int bb = valid ? n / G : 0, hg = valid ? n - bb * G : 0;
        cp_async16(qs + (ch >> 3) * q_panel + n * 128 + (((ch & 7) ^ (n & 7)) << 4),
                   qg + ((((size_t)nx.s * max_active + bb) * hq + (size_t)nx.g * G + hg) * D) / 8 + ch, valid);
    }
    if (smask_dst) {
        const uint64_t* src = mask + (size_t)nx.s * max_active * W;
        for (int idx = tid; idx < max_active * W; idx += NSOFT * 32) cp_async8(smask_dst + idx, src + idx);
    }
}

// The first pair's bitmaps and queries when the kernel runs ahead of the dependency wait (softmax
// threads; out of line, arguments by value).  The bitmaps are complete and are copied right away.
// The queries may still be written by the kernel ahead: their lines are only requested into L2
// (which stays coherent), the wait is taken, and then they are read and laid out as Q^T.
__device__ __noinline__ void stage_first_pair_early(const uint4* qg, const uint64_t* mask, int max_active, int W, int hq, int G, int s, int g, int M,
                                                    unsigned char* qs, int q_panel, uint64_t* smask_dst)
{
    const int tid = threadIdx.x;
    const int NP = (NP_MAX == 32 || M <= 32) ? 32 : ((NP_MAX == 64 || M <= 64) ? 64 : 128);
    if (smask_dst) {
        const uint64_t* src = mask + (size_t)s * max_active * W;
        for (int idx = tid; idx < max_active * W; idx += NSOFT * 32) smask_dst[idx] = src[idx];
    }
    for (int idx = tid * 8; idx < M * (D / 8); idx += NSOFT * 32 * 8) {      // one request per 128-byte line
        const int n = idx / (D / 8), ch = idx - n * (D / 8);
        const int bb = n / G, hg = n - bb * G;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(qg + ((((size_t)s * max_active + bb) * hq + (size_t)g * G + hg) * D) / 8 + ch));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int idx = tid; idx < NP * (D / 8); idx += NSOFT * 32) {
        const int n = idx / (D / 8), ch = idx - n * (D / 8);
        const bool valid = n < M;
        const int bb = valid ? n / G : 0, hg = valid ? n - bb * G : 0;
        cp_async16(qs + (ch >> 3) * q_panel + n * 128 + (((ch & 7) ^ (n & 7)) << 4),
                   qg + ((((size_t)s * max_active + bb) * hq + (size_t)g * G + hg) * D) / 8 + ch, valid);
    }
}

// Merge of the partials of one (scene, KV head) pair by the CTA that delivered the last one
// (all softmax threads).  Every thread owns four accumulator columns of one query row and merges
// the parts' (m, l, O) for them in ONE pass, three parts per turn with all loads ahead of the
// arithmetic (a turn costs one trip to L2; the running maximum is carried like in the online
// softmax, so more parts need no second pass):
//     m = max_c m_c,  l = sum_c l_c 2^(m_c - m),  O = sum_c O_c 2^(m_c - m) / l.
// Out of line, arguments by value.
__device__ __noinline__ void merge_pair(const float* ws_ml, const float* ws_o, __nv_bfloat16* out, int pair, int mmax, int M, int G, int s, int g,
                                        int max_active, int hq, int c_first, int c_last)
{
    constexpr int MB = 3;                          // parts per turn
    const int tid = threadIdx.x;
    __threadfence();
    for (int idx = tid; idx < M * (D / 4); idx += NSOFT * 32) {
        const int m = idx / (D / 4), c4 = idx - m * (D / 4);
        const float2* ml = reinterpret_cast<const float2*>(ws_ml + ((size_t)pair * mmax + m) * 2);
        const float4* po = reinterpret_cast<const float4*>(ws_o + ((size_t)pair * mmax + m) * D) + c4;
        const size_t cs = (size_t)mmax, os = (size_t)mmax * (D / 4);      // strides between CTAs' entries
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float mx = -INFINITY, lt = 0.f;
        for (int c0 = c_first; c0 <= c_last; c0 += MB) {
            float2 v[MB];
            float4 o[MB];
#pragma unroll
            for (int j = 0; j < MB; ++j) {
                const bool on = c0 + j <= c_last;
                v[j] = on ? __ldcg(ml + (size_t)(c0 + j) * cs) : make_float2(-INFINITY, 0.f);
                o[j] = on ? __ldcg(po + (size_t)(c0 + j) * os) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            float nm = mx;
#pragma unroll
            for (int j = 0; j < MB; ++j) nm = fmaxf(nm, v[j].x);
            const float sc = mx == nm ? 1.f : fast_exp2(mx - nm);           // (-inf) - (-inf) must not be formed
            lt *= sc;
            acc.x *= sc;
            acc.y *= sc;
            acc.z *= sc;
            acc.w *= sc;
#pragma unroll
            for (int j = 0; j < MB; ++j) {
                const float w = v[j].x == -INFINITY ? 0.f : fast_exp2(v[j].x - nm);   // a part that saw nothing
                lt = fmaf(v[j].y, w, lt);
                acc.x = fmaf(o[j].x, w, acc.x);
                acc.y = fmaf(o[j].y, w, acc.y);
                acc.z = fmaf(o[j].z, w, acc.z);
                acc.w = fmaf(o[j].w, w, acc.w);
            }
            mx = nm;
        }
        const float inv = 1.f / lt;
        const int b = m / G, hg = m - b * G;
        uint2 pk;
        pk.x = pack2(acc.x * inv, acc.y * inv);
        pk.y = pack2(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(out + (((size_t)s * max_active + b) * hq + (size_t)g * G + hg) * D + c4 * 4) = pk;
    }
}

// The rare path of the softmax, kept out of line so that the per-round loop stays small: the
// first round of a segment, or two (two groups: three) rounds after some score exceeded its column's reference by
// more than 2^16.  Column maxima of the round are gathered (shuffle transpose-reduce per warp,
// one shared-memory slot per row quadrant), references that are unset or too low are replaced,
// alpha[n] = 2^(old - new) is published, and the column sums (TMEM) and the accumulator O^T are
// rescaled where a reference moved.  Called by all softmax threads.  Returns 1 when a bounded
// wait ran out.  All arguments by value.
struct RaiseArgs {
    float* mneg;                 // column state in shared memory: mneg[128], alpha[128], lred[512], cmax[128], flags[4]
    volatile int* abortp;
    int32_t* status;
    uint32_t s_addr, o_addr;     // TMEM addresses of this thread's first score / accumulator column
    int np;                      // query columns of the pair, padded (32 / 64 / 128)
    uint32_t pv_bar, pv_parity;  // completion of the previous round's O^T += V^T P^T
    uint32_t vis;                // Eq. 1 bits of this thread's columns
    float c;
    int col0, nph;               // this thread's columns
    int live;                    // 1: the thread's KV row exists; 0: it does not (second half of a one-tile round); -1: the round
                                 // belongs to the other group of softmax warps, this one only takes part in the barriers
    int rescale_o, dead;
};
__device__ __noinline__ int raise_references(const RaiseArgs a)
{
    const int np = a.np;
    float* alpha = a.mneg + 128;
    int* wmax = reinterpret_cast<int*>(a.mneg + 256);      // [4][128]: maxima per row quadrant (shares the lred block)
    int* flags = reinterpret_cast<int*>(a.mneg + 768) + 128;
    const int tid = threadIdx.x, lane = threadIdx.x & 31, q4 = (threadIdx.x >> 5) & 3;
    bool dead = a.dead != 0;
    for (int ch = 0; ch < (a.live < 0 ? 0 : a.nph / 8); ++ch) {
        float mine = -INFINITY;                              // lane i < 8 ends up with the maximum of column ch * 8 + i
        if (a.live > 0) {
            uint32_t sv[8];
            tmem_ld<8>(a.s_addr + ch * 8, sv);
            tmem_wait_ld();
            float v[8];
            const uint32_t vb = a.vis >> (ch * 8);
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = ((vb >> i) & 1) ? __uint_as_float(sv[i]) * a.c : -INFINITY;
            // lanes whose index differs in bits >= 8 hold rows of the same columns: plain max
#pragma unroll
            for (int o = 16; o >= 8; o >>= 1)
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = fmaxf(v[i], __shfl_xor_sync(0xffffffffu, v[i], o));
            // transpose-reduce: at distance k a lane keeps the half of the columns that matches its bit k
#pragma unroll
            for (int k = 4; k >= 1; k >>= 1) {
                const bool up = (lane & k) != 0;
#pragma unroll
                for (int i = 0; i < k; ++i) {
                    const float recv = __shfl_xor_sync(0xffffffffu, up ? v[i] : v[i + k], k);
                    v[i] = fmaxf(up ? v[i + k] : v[i], recv);
                }
            }
            mine = v[0];
        }
        if (lane < 8) wmax[q4 * 128 + a.col0 + ch * 8 + lane] = ord_of(mine);
    }
    if (tid == 0) flags[0] = 0;
    raise_sync(smem_u32(const_cast<int*>(a.abortp)) - RAISE_BAR_BEFORE_ABORT_FLAG, a.abortp, a.status);
    if (tid < ((np + 31) & ~31)) {                         // whole warps (the shuffles below need all lanes)
        // highest column maximum of the round (every warp of these threads computes it for itself)
        int gm = INT_MIN;
        for (int n = lane; n < np; n += 32)
            gm = max(gm, max(max(wmax[n], wmax[128 + n]), max(wmax[256 + n], wmax[384 + n])));
#pragma unroll
        for (int o = 16; o; o >>= 1) gm = max(gm, __shfl_xor_sync(0xffffffffu, gm, o));
        if (tid < np) {
            const int m01 = max(wmax[tid], wmax[128 + tid]), m23 = max(wmax[256 + tid], wmax[384 + tid]);
            const float mx = ord_to(max(m01, m23));
            const float old = a.mneg[tid];                     // -reference, or UNSET
            float al = 1.f;
            if (old == UNSET) {
                // a column that sees no row yet borrows the round's highest reference: it will rarely have
                // to be raised later, and lower scores only make its terms smaller (far from underflow)
                const float ref = mx != -INFINITY ? mx : ord_to(gm);
                if (ref != -INFINITY) a.mneg[tid] = -ref;
            } else if (mx > RAISE_LOG2 - old) {
                al = fast_exp2(-old - mx);
                a.mneg[tid] = -mx;
                flags[0] = 1;
            }
            alpha[tid] = al;
        }
    }
    raise_sync(smem_u32(const_cast<int*>(a.abortp)) - RAISE_BAR_BEFORE_ABORT_FLAG, a.abortp, a.status);
    if (flags[0]) {                                        // a reference moved: rescale the accumulators (column sums and O^T)
        if (a.rescale_o) {
            if (!dead && !mbar_wait(a.pv_bar, a.pv_parity, a.abortp, a.status)) dead = true;   // no MMA may be writing O^T
            dead = __any_sync(0xffffffffu, dead);
            tc_fence_after();
            if (!dead) {
                for (int ch = 0; ch < a.nph / 8; ++ch) {
                    uint32_t ov[8];
                    tmem_ld<8>(a.o_addr + ch * 8, ov);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 8; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha[a.col0 + ch * 8 + i]);
                    tmem_st<8>(a.o_addr + ch * 8, ov);
                }
                if (a.col0 == 0) {                          // the column sums: TMEM lane n belongs to query column n
                    const uint32_t l_addr = a.o_addr - TM_O + TM_L;
                    uint32_t lv[8];
                    tmem_ld<8>(l_addr, lv);
                    tmem_wait_ld();
                    const float al = alpha[threadIdx.x & 127];
#pragma unroll
                    for (int i = 0; i < 8; ++i) lv[i] = __float_as_uint(__uint_as_float(lv[i]) * al);
                    tmem_st<8>(l_addr, lv);
                }
            }
        }
        tmem_wait_st();
    }
    return dead ? 1 : 0;
}

// The softmax warps' work on one segment; nphj = a quarter of the pair's padded query columns NP (8,
// 16 or 32).  Columns are handled eight at a time in real loops with the references read from
// shared memory, so that the same small loop serves every width.
//
// NGRP = 2 (launches whose widest pair has 33 to 64 query rows; measured: 3 to 6 % faster there, 1 %
// slower with fewer rows): the sixteen warps work as TWO GROUPS of eight on alternate rounds (group =
// round & 1: the round's score buffer and P^T buffer are then that group's own): a thread handles
// one KV row x NP / 2 columns of every other round, and while one group sits in the latency chain
// around a round (barrier tests, fences, arrivals) the other one is in its arithmetic.  Every warp
// still walks through all rounds of the segment, so both groups meet at the same places: the
// segment's set-up and end, its first round (references), its last round (next queries), and a
// raise of the references, which both decide on from a note that is three rounds old (by then it
// is final for either group without a wait of its own).
// NGRP = 1: all sixteen warps on every round, a thread handles one KV row x NP / 4 columns (with 128
// query rows there are two score buffers and one P^T buffer only).
__device__ __forceinline__ void softmax_segment(const AttnParams& p, const Ctx& cx, const Segment& sg, const int nph, const uint32_t seg,
                                                const long long hi, int& prefetched, uint32_t& g, int& vst, uint32_t& vph, bool& dead, const int warp, const int lane)
{
    const int np = NPART * nph;                   // the pair's padded query columns
    const int tid = threadIdx.x;                  // 0..NSOFT * 32 - 1
    const int q4 = warp & 3, part = warp >> 2;
    const int krow = q4 * 32 + lane;              // KV row of the round = TMEM lane of S^T; head_dim index for O^T
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    constexpr int ngrp = NGRP;                    // groups of softmax warps (two: warp >> 3 is the group, it works on the rounds of that parity)
    const int nphr = nph * ngrp, nchr = nphr >> 3;              // (round mapping: a group = 4 row quadrants x 4 / ngrp column parts)
    const int col0r = (ngrp == 2 ? (part & 1) : part) * nphr;
    const float c = p.scale_log2;
    const int A = cx.nact[sg.s];
    const int M = A * p.group;
    const int G = p.group;
    const int b_lo = col0r / G;                   // branch of this thread's first query column
    auto wait_u = [&](uint32_t bar, uint32_t parity) {    // warp-uniform outcome
        if (dead || __all_sync(0xffffffffu, mbar_try(bar, parity))) return;          // usually satisfied already
        if (!mbar_wait_slow(bar, parity, cx.abortp, p.status)) dead = true;
        dead = __any_sync(0xffffffffu, dead);
    };
    if (tid == 0 && seg == 0) FDC_TS(5);
    if (tid == 0) FDC_TSS(0);
    // ---- Q^T (B operand of S^T = K Q^T): row n = query row, K-major, 128B swizzle, rows >= M zero
    const bool published = prefetched == 2;       // Q^T, the bitmaps and their OR were completed and announced at the end of the previous segment
    {
        if (prefetched) {
            // queries and bitmaps were copied asynchronously during the previous segment's last round
            if (!published) cp_async_wait_all();
            prefetched = 0;
        } else {
            // all global reads first (one latency), then the stores
            const uint4* qg = reinterpret_cast<const uint4*>(p.q);
            constexpr int QPT = NP_MAX * (D / 8) / (NSOFT * 32);   // 16-byte chunks per thread for the widest pair of this build
            uint4 qv[QPT];
#pragma unroll
            for (int i = 0; i < QPT; ++i) {
                const int idx = tid + i * (NSOFT * 32);
                const int n = idx / (D / 8), ch = idx - n * (D / 8);
                qv[i] = make_uint4(0u, 0u, 0u, 0u);
                if (n < M) {
                    const int b = n / G, hg = n - b * G;
                    qv[i] = qg[((((size_t)sg.s * p.max_active + b) * p.hq + (size_t)sg.g * G + hg) * D) / 8 + ch];
                }
            }
            uint64_t mv[(NP_MAX > 64 ? MBUF_MAX : MBUF) / (NSOFT * 32)];
            const int nw = cx.mstaged ? p.max_active * p.W : 0;
#pragma unroll
            for (int i = 0; i < (NP_MAX > 64 ? MBUF_MAX : MBUF) / (NSOFT * 32); ++i) {
                const int idx = tid + i * (NSOFT * 32);
                mv[i] = idx < nw ? p.mask[(size_t)sg.s * p.max_active * p.W + idx] : 0ull;
            }
#pragma unroll
            for (int i = 0; i < QPT; ++i) {
                const int idx = tid + i * (NSOFT * 32);
                const int n = idx / (D / 8), ch = idx - n * (D / 8);
                if (n < np) *reinterpret_cast<uint4*>(cx.qs + (ch >> 3) * cx.q_panel + n * 128 + (((ch & 7) ^ (n & 7)) << 4)) = qv[i];
            }
#pragma unroll
            for (int i = 0; i < (NP_MAX > 64 ? MBUF_MAX : MBUF) / (NSOFT * 32); ++i) {
                const int idx = tid + i * (NSOFT * 32);
                if (idx < nw) cx.smask[(seg & 1) * cx.mbuf + idx] = mv[i];
            }
        }
        if (cx.mstaged && p.W <= UW && !published) {
            // OR of the scene's bitmaps: the rows that some branch may see (the others are cleared in V)
            soft_sync();                              // everybody's share of the bitmaps is in place
            if (tid < p.W) {
                const uint64_t* mb = cx.smask + (seg & 1) * cx.mbuf + tid;
                uint64_t un = 0ull;
                for (int b = 0; b < A; ++b) un |= mb[(size_t)b * p.W];
                cx.sunion[(seg & 1) * UW + tid] = un;
            }
        }
        if (tid < np) cx.mneg[tid] = UNSET;
        if (!published) {
            fence_async_smem();
            __syncwarp();
            if (!dead && lane == 0) mbar_arrive(cx.q_ready());
        }
        soft_sync();
        if (tid == 0 && seg == 0) FDC_TS(6);
        if (tid == 0) FDC_TSS(1);
    }

    const int ntile = sg.j1 - sg.j0;
    int t = 0;                                    // round within the segment
    for (int jb = 0; jb < ntile; jb += 32) {
        const int jn = ntile - jb < 32 ? ntile - jb : 32;
        const int my_tile = lane < jn ? p.tiles[(size_t)sg.s * p.ntile_max + sg.j0 + jb + lane] : 0;
        for (int k = 0; k < jn; k += 2, ++g, ++t) {
            const int nt = jn - k < 2 ? 1 : 2;
            const uint32_t b = g & 1;
            if (tid == 0) FDC_TR(g, 0);
            const int ti = q4 >> 1;                                   // which tile of the round this warp's rows are in
            const int tile = __shfl_sync(0xffffffffu, my_tile, (k + ti) & 31);
            const bool mine = ngrp == 1 || ((g ^ (uint32_t)(warp >> 3)) & 1u) == 0u;   // this warp's group works on the round (warps 0..7: even rounds)
            const bool live = mine && ti < nt && !dead;               // rows 64..127 of a one-tile round hold nothing
            const bool masked = live && tile * TILE + TILE > p.P;
            // Eq. 1 for this thread's KV row: bit i of vis <=> column col0r + i may see the row
            const uint32_t vis = masked ? row_visibility(mask_row(p, cx, seg, sg.s, 0), p.W, p.P, tile, (q4 & 1) * 32 + lane, A, G, b_lo, col0r, nphr) : ~0u;
            const uint32_t sb = g & (cx.ns - 1);                      // score buffer of the round
            const bool last_round = jb + k + 2 >= ntile && sg.next_u < hi;
            if (mine || last_round) {
                wait_u(cx.s_full() + 8 * sb, (g / cx.ns) & 1);
                tc_fence_after();
            }
            if (tid == 0) FDC_TR(g, 1);
            if (last_round) {
                // last round: every S^T = K Q^T of this segment has completed, so Q^T may be overwritten.
                // The next segment's queries (and its scene's bitmaps, into the other buffer) are copied
                // asynchronously; the latency hides behind this round, the drain and the partial write.
                prefetch_next_segment(reinterpret_cast<const uint4*>(p.q), p.mask, p.max_active, p.W, p.hq, G, p.hkv, cx.pre, cx.nact, cx.qs,
                                      cx.q_panel, cx.mstaged ? cx.smask + ((seg + 1) & 1) * cx.mbuf : nullptr, sg.next_u, hi, sg.s);
                prefetched = 1;
            }
            // The P^T buffer is still being read until the PV that used it last (two rounds ago, or the
            // previous round when there is a single buffer) has completed.  Past this wait every softmax
            // warp has also finished round g - 2 (one group), so what that round left in rflag is the same
            // for all.  With two groups only the round's own group waits; what both groups know without
            // any further wait is that round g - 3 is over for everybody (the owners of round g through
            // this wait, the others through theirs a round ago), so there a pending raise is looked for
            // three rounds after the note.  (No warp ever waits for a barrier of the other group's rounds
            // in mid-segment: a parity wait tells only two consecutive phases apart, and nothing would keep
            // that barrier from moving on twice.)
            if (mine) {
                if (cx.npb == 2) wait_u(cx.pv_done() + 8 * b, ((g >> 1) & 1) ^ 1);
                else if (g > 0) wait_u(cx.pv_done() + 8 * ((g - 1) & 1), ((g - 1) >> 1) & 1);
            }
            if (tid == 0) FDC_TR(g, 2);
            const uint32_t s_addr = cx.tmem + lane_base + sb * cx.s_stride + col0r;
            // References are set in the first round of a segment.  Later a score more than 2^16 above its
            // reference only leaves a note (no barrier in the common path): p stays far from overflow, and
            // two (two groups: three) rounds later, when all warps are known to see the note, the references are raised.
            if (t == 0 && __shfl_sync(0xffffffffu, my_tile, k & 31) * TILE + TILE <= p.P) {
                // First round of a segment inside the prefix: every column takes its score against the
                // round's first KV row (visible to all) as reference.  That row's own term is then exactly
                // 1, so no column sum can vanish; higher scores are handled by the lazy raise as usual.
                if (mine && q4 == 0 && !dead) {                       // the warps (of the round's group) that hold TMEM lane 0
#pragma unroll 1
                    for (int ch = 0; ch < nchr; ++ch) {
                        uint32_t sv[8];
                        tmem_ld<8>(s_addr + ch * 8, sv);
                        tmem_wait_ld();
                        if (lane == 0) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) cx.mneg[col0r + ch * 8 + i] = -(__uint_as_float(sv[i]) * c);
                        }
                    }
                }
                soft_sync();
            } else if (t == 0 || (NGRP == 1 ? (g >= 2 && cx.rflag[(g - 2) & 7] == (int)(g - 2)) : (t >= 3 && cx.rflag[(g - 3) & 7] == (int)(g - 3)))) {
                RaiseArgs ra;
                ra.mneg = cx.mneg;
                ra.abortp = cx.abortp;
                ra.status = p.status;
                ra.s_addr = s_addr;
                ra.o_addr = cx.tmem + lane_base + TM_O + col0r;
                ra.np = np;
                ra.pv_bar = cx.pv_done() + 8 * ((g - 1) & 1);
                ra.pv_parity = ((g - 1) >> 1) & 1;
                ra.vis = vis;
                ra.c = c;
                ra.col0 = col0r;
                ra.nph = nphr;
                ra.live = mine ? (live ? 1 : 0) : -1;
                ra.rescale_o = mine && t > 0;
                ra.dead = dead;
                dead = raise_references(ra) != 0;
            }
            if (tid == 0) FDC_TR(g, 3);
            if (!mine) {                                              // the other group's round
                if (++vst == cx.nv) {
                    vst = 0;
                    vph ^= 1;
                }
                continue;
            }
            if (live) {
                unsigned char* prow = cx.ps + (b & (cx.npb - 1)) * cx.p_buf + krow * 128;
                float emax = 0.f;
#pragma unroll 1
                for (int ch = 0; ch < nchr; ++ch) {
                    uint32_t sv[8];
                    tmem_ld<8>(s_addr + ch * 8, sv);
                    const float4 m0 = *reinterpret_cast<const float4*>(cx.mneg + col0r + ch * 8);
                    const float4 m1 = *reinterpret_cast<const float4*>(cx.mneg + col0r + ch * 8 + 4);
                    const float mn[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
                    tmem_wait_ld();
                    if (masked) {                                      // uniform branch: prefix rounds skip the selects
                        const uint32_t vb = vis >> (ch * 8);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (!((vb >> i) & 1)) sv[i] = 0xff800000u;
                    }
                    float e[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        e[i] = fast_exp2(fmaf(__uint_as_float(sv[i]), c, mn[i]));
                        emax = fmaxf(emax, e[i]);
                    }
                    // P^T goes to the tensor core as bf16.  The column sums (the softmax denominators) are taken by
                    // the tensor core too, from the SAME rounded values (a multiplication of P^T by ones beside
                    // every O^T += V^T P^T), so numerator and denominator stay consistent: the rounding cancels
                    // where a few terms dominate.
                    uint32_t pk[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) pk[j] = pack2(e[2 * j], e[2 * j + 1]);
                    const int cidx = (col0r >> 3) + ch;                // 16-byte chunk of the P^T row
                    *reinterpret_cast<uint4*>(prow + (cidx >> 3) * PANEL + (((cidx & 7) ^ (krow & 7)) << 4)) =
                        make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
                if (emax > 65536.f) {                                  // 2^16 above the reference: note it for round g + 2
                    cx.rflag[g & 7] = (int)g;
                    if (!(emax < 1.0e30f)) atomicOr(p.status, FDC_DEV_SCORE_RANGE);     // beyond 2^100 (or inf / nan)
                }
            }
            if (tid == 0) FDC_TR(g, 4);
            // ---- this round's V stage.  Beyond the prefix, rows that no branch of the scene may see can hold
            // anything (NaN, Inf: slots that were never written), and although their P^T entries are
            // exactly 0, 0 * NaN must not reach the accumulator.  The multiplication runs in steps of 16
            // KV rows: a step without any visible row is left out, and in the other steps the unseen
            // rows are cleared here, every thread a quarter of its own row, once the stage has landed.
            uint32_t st4 = live ? 0xfu : 0u;                           // steps of this warp's tile to multiply
            if (masked) {                                              // (uniform over the warp)
                const uint64_t* un = (cx.mstaged && p.W <= UW) ? cx.sunion + (seg & 1) * UW : nullptr;
                const int w = tile - p.P / TILE;
                const uint64_t seen = (un && (p.P & (TILE - 1)) == 0) ? (w < p.W ? un[w] : 0ull)
                                                                       : tile_seen_rows(un, mask_row(p, cx, seg, sg.s, 0), p.W, p.P, A, tile);
                wait_u(cx.v_full() + 8 * vst, vph);
                const int row = (q4 & 1) * 32 + lane;
                const bool none = seen == 0ull;                        // (such a tile should not be listed: clear and multiply all of it)
                const uint32_t step_seen = (uint32_t)(seen >> (row & 48)) & 0xffffu;
                if (!dead && (none || (step_seen != 0u && !((seen >> row) & 1ull)))) {
                    // the column parts of the group share the row's 256 bytes (two panels of 128): a quarter each, or a half
                    if constexpr (NGRP == 1) {
                        const uint32_t va = smem_u32(cx.vring) + (uint32_t)vst * STAGE + (uint32_t)(part >> 1) * PANEL +
                                            (uint32_t)(ti * TILE + row) * 128 + (uint32_t)(part & 1) * 64;
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(va + (uint32_t)((i + lane) & 3) * 16), "r"(0u) : "memory");
                    } else {
                        const uint32_t va = smem_u32(cx.vring) + (uint32_t)vst * STAGE + (uint32_t)(part & 1) * PANEL + (uint32_t)(ti * TILE + row) * 128;
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(va + (uint32_t)((i + lane) & 7) * 16), "r"(0u) : "memory");
                    }
                }
                st4 = 0u;
#pragma unroll
                for (int i = 0; i < 4; ++i) st4 |= (none || ((seen >> (16 * i)) & 0xffffull)) ? (1u << i) : 0u;
                // the whole tiles of the prefix come first in a tile list (entry j = tile j): the producer relies on it
                if (col0r == 0 && (q4 & 1) == 0 && lane == 0 && sg.j0 + jb + k + ti < p.P / TILE) atomicOr(p.status, FDC_DEV_TILE_LIST);
            }
            if (col0r == 0 && (q4 & 1) == 0 && lane == 0) cx.v_steps[b * 2 + ti] = (int)st4;
            if (++vst == cx.nv) {
                vst = 0;
                vph ^= 1;
            }
            // every thread orders its own TMEM reads and shared-memory writes, then one lane per warp signals
            tc_fence_before();
            fence_async_smem();
            __syncwarp();
            if (!dead && lane == 0) {
                mbar_arrive(cx.s_free() + 8 * sb);                       // the scores have been read: K Q^T may reuse the buffer
                mbar_arrive(cx.p_full() + 8 * b);
            }
            if (tid == 0) FDC_TR(g, 5);
        }
    }
    if (tid == 0) { FDC_TS(7); FDC_TSS(2); }
    if (prefetched == 1) {
        // The next pair's queries are announced before this pair is finished off, so that its K Q^T runs
        // on (into the score buffers) while the last multiplications drain and the result is written.
        cp_async_wait_all();
        if (cx.mstaged && p.W <= UW) {
            soft_sync();
            int s2 = sg.s;
            const Segment nx = decode_segment(sg.next_u, hi, cx.pre, p.hkv, s2);
            if (tid < p.W) {
                const uint64_t* mb = cx.smask + ((seg + 1) & 1) * cx.mbuf + tid;
                uint64_t un = 0ull;
                const int A2 = cx.nact[nx.s];
                for (int b = 0; b < A2; ++b) un |= mb[(size_t)b * p.W];
                cx.sunion[((seg + 1) & 1) * UW + tid] = un;
            }
        }
        fence_async_smem();
        __syncwarp();
        if (!dead && lane == 0) mbar_arrive(cx.q_ready());
        prefetched = 2;
    }
    // ---- end of segment: the accumulator is final once the last PV has completed
    // (joint mapping from here on: sixteen warps = 4 row quadrants x 4 column parts)
    const int nch = nph >> 3, col0 = part * nph;
    const uint32_t o_addr = cx.tmem + lane_base + TM_O + col0;
    // A parity wait only tells two consecutive phases of a barrier apart, so a warp may wait for a
    // round's completion only when it knows the round two before to be complete.  The group whose
    // round the last one was not has not looked at that round's barrier for a while: it first waits
    // for the round before (its own, or the one it knows the predecessor of), which brings it close
    // enough.
    const uint32_t last = g - 1;
    if (ngrp == 2 && t > 1) wait_u(cx.pv_done() + 8 * ((last - 1) & 1), ((last - 1) >> 1) & 1);
    wait_u(cx.pv_done() + 8 * (last & 1), (last >> 1) & 1);
    tc_fence_after();
    if (tid == 0) { FDC_TS(8); FDC_TSS(3); }
    // column sums: TMEM lane n of the accumulator of the multiplication by ones
    if (part == 0) {
        uint32_t lv[8];
        tmem_ld<8>(cx.tmem + lane_base + TM_L, lv);
        tmem_wait_ld();
        cx.lred[krow] = __uint_as_float(lv[0]);
    } else {
        cx.lred[part * 128 + krow] = 0.f;
    }
    soft_sync();
    const int pair = sg.s * p.hkv + sg.g;
    const int slot = blockIdx.x + pair;
    const bool whole = sg.j0 == 0 && sg.j1 == sg.nt;       // this CTA saw every tile of the pair
    if (tid == 0) FDC_TSS(4);
    if (p.pair_cnt && whole) {
        // no other partial exists: normalise and write the output directly
        if (tid < np) cx.alpha[tid] = 1.f / ((cx.lred[tid] + cx.lred[128 + tid]) + (cx.lred[256 + tid] + cx.lred[384 + tid]));
        soft_sync();
        if (!dead) {
            __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out);
#pragma unroll 1
            for (int ch = 0; ch < nch; ++ch) {
                uint32_t ov[8];
                tmem_ld<8>(o_addr + ch * 8, ov);
                tmem_wait_ld();
                int b = (col0 + ch * 8) / G, hg = (col0 + ch * 8) - b * G;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int n = col0 + ch * 8 + i;
                    if (n < M)
                        out[(((size_t)sg.s * p.max_active + b) * p.hq + (size_t)sg.g * G + hg) * D + krow] =
                            __float2bfloat16_rn(__uint_as_float(ov[i]) * cx.alpha[n]);
                    if (++hg == G) {
                        hg = 0;
                        ++b;
                    }
                }
            }
        }
    } else {
        if (!dead) {
            if (tid < M) {
                const float lt = (cx.lred[tid] + cx.lred[128 + tid]) + (cx.lred[256 + tid] + cx.lred[384 + tid]);
                const float mn = cx.mneg[tid];
                *reinterpret_cast<float2*>(p.ws_ml + ((size_t)slot * p.mmax + tid) * 2) = make_float2(mn == UNSET ? -INFINITY : -mn, lt);
            }
            // O^T: lane = head_dim index, column = query row; partials are stored [query row][head_dim]
            float* wo = p.ws_o + (size_t)slot * p.mmax * D + krow;
#pragma unroll 1
            for (int ch = 0; ch < nch; ++ch) {
                uint32_t ov[8];
                tmem_ld<8>(o_addr + ch * 8, ov);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (col0 + ch * 8 + i < M) wo[(size_t)(col0 + ch * 8 + i) * D] = __uint_as_float(ov[i]);
            }
        }
        if (tid == 0) FDC_TSS(5);
        if (p.pair_cnt) {
            // the CTA that delivers the last partial of a pair merges them all (no second kernel)
            __threadfence();
            soft_sync();
            if (tid == 0) {
                int c_first, c_last;
                pair_ctas(p, cx, sg.s, sg.g, c_first, c_last);
                const int expected = c_last - c_first + 1;               // every CTA in between owns tiles of the pair
                const int old = dead ? -1 : atomicAdd(&p.pair_cnt[pair], 1);
                cx.flags[1] = old == expected - 1;
                cx.flags[2] = c_first;
                cx.flags[3] = c_last;
                if (old == expected - 1) p.pair_cnt[pair] = 0;          // ready for the next call
            }
            soft_sync();
            if (tid == 0) FDC_TSS(6);
            if (cx.flags[1])
                merge_pair(p.ws_ml, p.ws_o, reinterpret_cast<__nv_bfloat16*>(p.out), pair, p.mmax, M, G, sg.s, sg.g, p.max_active, p.hq,
                           cx.flags[2], cx.flags[3]);
        }
    }
    soft_sync();                     // column state and Q^T are free again
    if (tid == 0) { FDC_TS(9); FDC_TSS(8); }
    tc_fence_before();
    __syncwarp();
    if (!dead && lane == 0) mbar_arrive(cx.o_free());
}

__global__ void __launch_bounds__(THREADS, 1)
FDC_TC_KERNEL(const AttnParams p, const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const int nk, const int nv, const int split_only)
{
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_dyn + 1023) & ~(uintptr_t)1023);
    Ctx cx;
    cx.nk = nk;
    cx.nv = nv;
    constexpr int np_max = NP_MAX, npb = NP_MAX > 64 ? 1 : 2;      // (128 query rows: one P^T buffer, so that four stages still fit)
    cx.q_panel = np_max * 128;
    cx.p_buf = ((np_max + 63) / 64) * PANEL;
    // (register allocation: with this one value folded into the address arithmetic the two wider builds
    // spill; kept in a register they do not, or hardly)
    if (NP_MAX > 32) asm volatile("" : "+r"(cx.p_buf));
    cx.npb = npb;
    cx.kring = smem;
    cx.vring = cx.kring + (size_t)nk * STAGE;
    cx.ps = cx.vring + (size_t)nv * STAGE;
    cx.qs = cx.ps + npb * cx.p_buf;
    cx.ones = cx.qs + (D / 64) * cx.q_panel;
    uint64_t* bars = reinterpret_cast<uint64_t*>(cx.ones + ONES_BYTES);
    cx.bar0 = smem_u32(bars);
    cx.ns = np_max <= 64 ? 4 : 2;
    cx.s_stride = np_max <= 64 ? 64 : 128;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 5 * MAXST + 16);
    cx.mneg = reinterpret_cast<float*>(tmem_holder + 4);
    cx.alpha = cx.mneg + 128;
    cx.lred = cx.alpha + 128;
    cx.cmax = reinterpret_cast<int*>(cx.lred + 512);
    cx.flags = cx.cmax + 128;
    cx.rflag = cx.flags + 4;
    cx.pre = cx.rflag + 8;
    cx.nact = cx.pre + p.batch + 1;
    cx.prev = cx.nact + p.batch;
    cx.smask = reinterpret_cast<uint64_t*>(((uintptr_t)(cx.prev + p.batch + 1) + 15) & ~(uintptr_t)15);
    cx.mbuf = np_max > 64 ? MBUF_MAX : MBUF;
    cx.sunion = cx.smask + 2 * cx.mbuf;
    cx.mstaged = p.max_active * p.W <= cx.mbuf;
    __shared__ CtaFlags cta_flags;
    cx.abortp = &cta_flags.abort_flag;
    cx.v_steps = cta_flags.v_steps;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) FDC_TS(0);
    if (threadIdx.x == 0) {
        cta_flags.abort_flag = 0;
    }
    if (threadIdx.x < 8) cx.rflag[threadIdx.x] = -1;
    if (threadIdx.x < ONES_BYTES / 4 && !split_only) {
        reinterpret_cast<uint32_t*>(cx.ones)[threadIdx.x] = 0x3F803F80u;          // bf16 1.0 twice
        fence_async_smem();
    }
    // The layers of one forward pass see the same per-scene counts, so the work split is made once
    // per pass (a launch of this kernel with split_only set) and kept in the memo, with the counts it
    // was computed from.  The memo's loads and those of the counts are all issued before the first
    // use, so that they share one trip to memory; when they may be read ahead of the dependency wait
    // they are issued right here, and the trip hides behind the set-up.
    constexpr int MEMO_MAGIC = 0x5D180000 | (W_PREFIX << 12) | (W_MASKED << 8) | W_PAIR;
    const int32_t* mrd = (p.split_memo && !split_only) ? p.split_memo : nullptr;
    int4 mh0 = make_int4(0, 0, 0, 0), mh1 = mh0, mh2 = mh0, me = mh0;
    int m_na = -1, m_nt = -1, m_prev = 0;
    int na[4], nt[4];
    auto issue_loads = [&]() {
        if (mrd) {
            mh0 = __ldcg(reinterpret_cast<const int4*>(mrd));
            mh1 = __ldcg(reinterpret_cast<const int4*>(mrd) + 1);
            mh2 = __ldcg(reinterpret_cast<const int4*>(mrd) + 2);
            me = __ldcg(reinterpret_cast<const int4*>(mrd + FDC_MEMO_ENTRIES) + blockIdx.x);
            if ((int)threadIdx.x < p.batch) {
                m_na = __ldcg(mrd + 16 + threadIdx.x);
                m_nt = __ldcg(mrd + 16 + FDC_MEMO_BATCH + threadIdx.x);
            }
            if ((int)threadIdx.x <= p.batch) m_prev = __ldcg(mrd + 16 + 2 * FDC_MEMO_BATCH + threadIdx.x);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = threadIdx.x + j * THREADS;
            na[j] = i < p.batch ? p.n_active[i] : 0;
            nt[j] = i < p.batch ? p.ntiles[i] : 0;
        }
    };
    if (p.early) issue_loads();
    // ---- set-up that needs no global memory: barriers, TMEM
    if (threadIdx.x == 0) {
        for (int i = 0; i < MAXST; ++i) {
            mbar_init(cx.k_full() + 8 * i, 1);
            mbar_init(cx.k_empty() + 8 * i, 1);
            mbar_init(cx.v_full() + 8 * i, 1);
            mbar_init(cx.v_empty() + 8 * i, 1);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(cx.s_full() + 8 * i, 1);
            mbar_init(cx.s_free() + 8 * i, NSOFT / NGRP);      // the warps of the round's group
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(cx.p_full() + 8 * i, NSOFT / NGRP);
            mbar_init(cx.pv_done() + 8 * i, 2);              // the V multiplications and the column sums
        }
        mbar_init(cx.q_ready(), NSOFT);
        mbar_init(cx.o_free(), NSOFT);
        mbar_init(cx.app_done(), 1);
        mbar_init(smem_u32(&cta_flags.raise_bar), NSOFT);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == W_QK && !split_only) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)), "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = split_only ? 0u : *reinterpret_cast<volatile uint32_t*>(tmem_holder);
    cx.tmem = tmem;
    if (threadIdx.x == 0) FDC_TS(1);
    // Programmatic dependent launch: this grid may have been scheduled while the kernel before it in
    // the stream was still running, and the kernel after this one may be scheduled early in the same
    // way.  Ordinarily nothing of global memory is touched before the kernel ahead has completed, and
    // only then is the next one let in.  With p.early the host vouches that the pass tables (counts,
    // tile lists, bitmaps), the work split and the prefix rows of the cache were complete before the
    // kernel ahead even began: then the work split is looked up and the first K/V stages of the prefix
    // are requested right away, while that kernel's last blocks are still running, and only what it
    // may have written (queries, the pass's new K/V rows, the rows beyond the prefix) waits for it.
    // Every thread passes the wait before the block ends, so grids complete in stream order.
    if (!p.early) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) FDC_TS(2);
    if (!p.early) issue_loads();
    bool active = true;                       // this CTA has units (uniform over the CTA)
    long long lo = 0, hi = 0;
    // the raw tile counts wait in prev[] for the scan
    {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = threadIdx.x + j * THREADS;
            if (i < p.batch) {
                cx.nact[i] = na[j];
                cx.prev[i] = nt[j];
            }
        }
        for (int i = threadIdx.x + 4 * THREADS; i < p.batch; i += THREADS) {
            cx.nact[i] = p.n_active[i];
            cx.prev[i] = p.ntiles[i];
        }
    }
    __syncthreads();
    const long long total = scan_ntiles(cx.prev, p.batch, cx.pre);
    const long long U = total * p.hkv;
    if (threadIdx.x == 0) FDC_TS(3);
    if (U == 0) active = false;
    cx.tpart = 0;
    cx.n_cta = p.n_cta;
    cx.vtot = 0;
    cx.npre = p.P / TILE;
    bool hit = false;
    if (mrd) {
        int same = mh0.x == MEMO_MAGIC && mh0.y == (int)p.seq && mh0.z == p.hkv && mh0.w == p.n_cta && mh1.x == p.P && mh1.y == p.batch;
        if ((int)threadIdx.x < p.batch) same = same && m_na == cx.nact[threadIdx.x] && m_nt == cx.pre[threadIdx.x + 1] - cx.pre[threadIdx.x];
        hit = __syncthreads_and(same) != 0;
    }
    if (hit) {
        // same counts as the launch before: its split stands
        cx.tpart = mh1.z;
        cx.n_cta = mh1.w;
        cx.vtot = ((long long)mh2.y << 32) | (uint32_t)mh2.x;
        if ((int)threadIdx.x <= p.batch) cx.prev[threadIdx.x] = m_prev;
        __syncthreads();
        lo = ((long long)me.y << 32) | (uint32_t)me.x;
        hi = ((long long)me.w << 32) | (uint32_t)me.z;
    } else if (!active) {
    } else if (p.pair_cnt) {
        // This kernel also merges the partial results of a pair.  Ending one pair and starting the
        // next inside a CTA costs as much as streaming a dozen tiles (drain, partial write, merge,
        // new queries), so while there are no more pairs than CTAs every CTA gets ONE part of ONE
        // pair: pairs are cut into the fewest equal parts of at most tpart (weighted) tiles, tpart the smallest
        // size (at least MIN_UNITS) for which the parts do not outnumber the CTAs.  With more pairs
        // than CTAs, CTAs get equal shares of a weighted length (see above).
        cx.npre = p.P / TILE;
        __shared__ int split_tpart, split_max, split_pairs;
        if (threadIdx.x == 0) {
            split_tpart = 0x7fffffff;
            split_max = 0;
            split_pairs = 0;
        }
        __syncthreads();
        {
            int nsc = 0, mx = 0;
            for (int i = threadIdx.x; i < p.batch; i += THREADS) {
                const int nt = cx.pre[i + 1] - cx.pre[i];
                nsc += nt > 0;
                mx = nt > mx ? nt : mx;
            }
            if (nsc) {
                atomicAdd(&split_pairs, nsc);
                atomicMax(&split_max, mx);
            }
        }
        __syncthreads();
#ifdef FDC_EQUAL_SHARES
        const bool one_part = false;                   // (development builds: always equal shares of the weighted length)
#else
        const bool one_part = (long long)split_pairs * p.hkv <= p.n_cta;
#endif
        if (one_part) {
            // every thread tries sizes of its own; the smallest that fits wins
            const uint32_t vmax = (uint32_t)vt_of(cx, split_max, split_max);
            const uint32_t tl = vmax < (uint32_t)MIN_UNITS ? vmax : (uint32_t)MIN_UNITS;
            const uint32_t budget = (uint32_t)(p.n_cta / p.hkv);          // parts per KV head
            for (uint32_t T = tl + threadIdx.x; T <= vmax && T < (uint32_t)split_tpart; T += THREADS) {
                uint32_t cnt = 0;
                for (int i = 0; i < p.batch; ++i) {
                    const int nt = cx.pre[i + 1] - cx.pre[i];
                    cnt += ((uint32_t)vt_of(cx, nt, nt) + T - 1) / T;
                }
                if (cnt <= budget) {
                    atomicMin(&split_tpart, (int)T);
                    break;
                }
            }
        } else if (threadIdx.x == 0) {
            split_tpart = 0;
        }
        __syncthreads();
        if (one_part && threadIdx.x == 0) {
            // One part per CTA leaves CTAs idle when the parts per pair do not divide the CTAs evenly
            // (64 pairs on 148 CTAs: 2 or 3 parts, a CTA carries up to 16 % more than the average).  Where the
            // shares are long enough for a pair boundary inside a CTA to cost less than that (measured:
            // from about 200 prefix tiles per CTA, half of that with 128 query rows, whose rounds take twice
            // as long), equal shares of the weighted length win after all.
            long long tot = 0;
            for (int i = 0; i < p.batch; ++i) {
                const int nt = cx.pre[i + 1] - cx.pre[i];
                if (nt > 0) tot += vt_of(cx, nt, nt) + W_PAIR;
            }
            const long long avg = tot * p.hkv / p.n_cta;
            if (avg * (np_max > 64 ? 2 : 1) >= 200 * W_PREFIX && (long long)split_tpart * 100 > avg * 108) split_tpart = 0;
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            const uint32_t T = (uint32_t)split_tpart;
            int carry = 0;
            for (int b0 = 0; b0 < p.batch; b0 += 32) {
                const int i = b0 + threadIdx.x;
                int x = 0;
                if (i < p.batch) {
                    const int nt = cx.pre[i + 1] - cx.pre[i];
                    x = T ? (int)(((uint32_t)vt_of(cx, nt, nt) + T - 1) / T) : (nt > 0 ? vt_of(cx, nt, nt) + W_PAIR : 0);
                }
                int inc = x;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(0xffffffffu, inc, o);
                    if ((int)threadIdx.x >= o) inc += y;
                }
                if (i < p.batch) cx.prev[i] = carry + inc - x;
                carry += __shfl_sync(0xffffffffu, inc, 31);
            }
            if (threadIdx.x == 0) cx.prev[p.batch] = carry;
        }
        __syncthreads();
        cx.tpart = split_tpart;
        if (cx.tpart) {
            const int c = blockIdx.x;
            cx.n_cta = cx.prev[p.batch] * p.hkv;
            if (c < cx.n_cta) {
                int sl = 0, sh = p.batch;              // largest s with prev[s] * hkv <= c
                while (sh - sl > 1) {
                    const int mid = (sl + sh) >> 1;
                    if (cx.prev[mid] * p.hkv <= c) sl = mid;
                    else sh = mid;
                }
                while (cx.prev[sl + 1] == cx.prev[sl]) ++sl;          // scenes without tiles have no parts
                const int k = cx.prev[sl + 1] - cx.prev[sl], nt = cx.pre[sl + 1] - cx.pre[sl];
                const uint32_t idx = (uint32_t)(c - cx.prev[sl] * p.hkv), g = idx / (uint32_t)k, i = idx - g * (uint32_t)k;
                const uint32_t V = (uint32_t)vt_of(cx, nt, nt);       // part i: tiles whose weighted start lies in [i V / k, (i + 1) V / k)
                const int j0 = tile_of_vt(cx, nt, (int)((i * V + k - 1) / (uint32_t)k));
                const int j1 = tile_of_vt(cx, nt, (int)(((i + 1) * V + k - 1) / (uint32_t)k));
                lo = (long long)cx.pre[sl] * p.hkv + (long long)g * nt + j0;
                hi = lo + (j1 - j0);
            }
        } else {
            const long long want = (U + MIN_TILES - 1) / MIN_TILES;      // small problems use fewer CTAs
            if (want < cx.n_cta) cx.n_cta = (int)want;
            cx.vtot = (long long)cx.prev[p.batch] * p.hkv;
            lo = unit_of_virt(p, cx, cta_first_unit(blockIdx.x, cx.vtot, cx.n_cta));
            hi = unit_of_virt(p, cx, cta_first_unit(blockIdx.x + 1, cx.vtot, cx.n_cta));
        }
    } else {
        cx.prev = nullptr;
        lo = cta_first_unit(blockIdx.x, U, cx.n_cta);
        hi = cta_first_unit(blockIdx.x + 1, U, cx.n_cta);
    }
    if (lo >= hi || (int)blockIdx.x >= cx.n_cta) active = false;
    if (threadIdx.x == 0) FDC_TS(4);
    if (split_only) {
        // this launch only computes the split and leaves it to the attention launches of the pass
        int32_t* mwr = p.split_memo;
        if (threadIdx.x == 0)
            reinterpret_cast<int4*>(mwr + FDC_MEMO_ENTRIES)[blockIdx.x] =
                active ? make_int4((int)(uint32_t)lo, (int)(lo >> 32), (int)(uint32_t)hi, (int)(hi >> 32)) : make_int4(0, 0, 0, 0);
        if (blockIdx.x == 0) {
            if (threadIdx.x == 0) {
                reinterpret_cast<int4*>(mwr)[0] = make_int4(MEMO_MAGIC, (int)p.seq, p.hkv, p.n_cta);
                reinterpret_cast<int4*>(mwr)[1] = make_int4(p.P, p.batch, cx.tpart, cx.n_cta);
                reinterpret_cast<int4*>(mwr)[2] = make_int4((int)(uint32_t)cx.vtot, (int)(cx.vtot >> 32), 0, 0);
            }
            if ((int)threadIdx.x < p.batch) {
                mwr[16 + threadIdx.x] = cx.nact[threadIdx.x];
                mwr[16 + FDC_MEMO_BATCH + threadIdx.x] = cx.pre[threadIdx.x + 1] - cx.pre[threadIdx.x];
            }
            if ((int)threadIdx.x <= p.batch) mwr[16 + 2 * FDC_MEMO_BATCH + threadIdx.x] = U > 0 ? cx.prev[threadIdx.x] : 0;
        }
    }

    if (split_only) active = false;
    // Two roles run ahead of the dependency wait (with p.early): the TMA producer, which takes the wait
    // itself once nothing more of the prefix can be requested, and the softmax warps, which first stage
    // the first pair's bitmaps.
    if (p.early && !(active && (warp == W_PROD || warp < NSOFT))) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!active) {
    } else if (warp == W_PROD) {
        producer_loop(p, cx, &tm_k, &tm_v, lo, hi, lane);
    } else if (warp == W_AUX) {
        aux_loop(p, cx, lo, hi, lane);
    } else if (warp == W_PV) {
        pv_loop(p, cx, lo, hi, lane);
    } else if (warp == W_QK) {
        qk_loop(p, cx, lo, hi, lane);
    } else {
        int s = 0;
        uint32_t g = 0, seg = 0;
        int vst = 0;                              // V ring stage and phase of round g
        uint32_t vph = 0;
        long long u = lo;
        bool dead = false;                        // a bounded wait ran out somewhere in the CTA
        int prefetched = 0;                       // the segment's queries and bitmaps are already on their way
        if (p.early) {
            // ahead of the dependency wait: the first pair's bitmaps; its queries follow right after the wait
            int s0 = 0;
            const Segment sg = decode_segment(lo, hi, cx.pre, p.hkv, s0);
            stage_first_pair_early(reinterpret_cast<const uint4*>(p.q), p.mask, p.max_active, p.W, p.hq, p.group, sg.s, sg.g,
                                   cx.nact[sg.s] * p.group, cx.qs, cx.q_panel, cx.mstaged ? cx.smask : nullptr);
            prefetched = 1;
        }
        while (u < hi) {
            const Segment sg = decode_segment(u, hi, cx.pre, p.hkv, s);
            const int M = cx.nact[sg.s] * p.group;
            softmax_segment(p, cx, sg, ((NP_MAX == 32 || M <= 32) ? 32 : ((NP_MAX == 64 || M <= 64) ? 64 : 128)) / NPART, seg, hi, prefetched, g, vst, vph, dead, warp, lane);
            ++seg;
            u = sg.next_u;
        }
    }
    // ---- teardown: everybody is done with TMEM before it is freed
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) FDC_TS(10);
    if (warp == W_QK && !split_only) {
        // TMEM is freed only when no multiplication can still be writing it.  In an orderly run they were
        // all seen to complete before the last result was written.  After a wait that ran out, some may
        // still be on their way: their operands are all on chip, so they finish within microseconds, and
        // the block lingers for about a hundred before it lets go of TMEM.
        if (*cx.abortp)
            for (int i = 0; i < 100; ++i) __nanosleep(1000);
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace

#ifdef FDC_TRACE
extern "C" int FDC_TC_TRACE_READ(long long* out)
{
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(out, g_tr, sizeof(long long) * 1024);
    cudaMemcpyFromSymbol(out + 1024, g_ts, sizeof(long long) * 80);
    return 0;
}
#endif

namespace fdc {

// bf16, head_dim 128, at most 128 query rows per (scene, KV head); FDC_ERR_SHAPE otherwise (the
// caller then takes another kernel).  split_only: the launch only computes the work split of the
// pass into p.split_memo (an ordinary launch; no rings, no TMEM).  This build of the kernel
// serves the launches whose widest pair has 33 to 64 query rows (two groups) or all others (one).
int FDC_TC_LAUNCH(const AttnParams& p, int head_dim, cudaStream_t st, int split_only)
{
    if (head_dim != D || p.mmax > 128) return FDC_ERR_SHAPE;
    const int np_max = p.mmax <= 32 ? 32 : (p.mmax <= 64 ? 64 : 128);
    const int p_buf = ((np_max + 63) / 64) * PANEL;
    if (np_max != NP_MAX) return FDC_ERR_SHAPE;   // another build's launches
    const int npb = np_max > 64 ? 1 : 2;          // 128 query rows: one P^T buffer, so that four stages still fit
    const size_t fixed = 1024 + (size_t)npb * p_buf + (size_t)(D / 64) * np_max * 128 + ONES_BYTES + 8 * (5 * MAXST + 16) + 16 +
                         4 * (128 + 128 + 512 + 128 + 12) + sizeof(int) * (3 * p.batch + 2) + 8 * (2 * (np_max > 64 ? MBUF_MAX : MBUF) + 2 * UW + 2) + 64;
    int stages = (int)((227 * 1024 - 256 - fixed) / STAGE);
    if (stages > 2 * MAXST) stages = 2 * MAXST;
    if (stages < 4) return FDC_ERR_SHAPE;
    if (split_only) stages = 0;
    const int nk = stages / 2, nv = stages - nk;
    const size_t smem = fixed + (size_t)stages * STAGE;
    alignas(64) CUtensorMap tk, tv;
    int rc = get_kv_tensor_map(p.k, p, D, TILE, &tk);
    if (rc) return rc;
    rc = get_kv_tensor_map(p.v, p, D, TILE, &tv);
    if (rc) return rc;
    static size_t attr_smem[kMaxDevices] = {};
    rc = raise_dynamic_smem(reinterpret_cast<const void*>(FDC_TC_KERNEL), smem, attr_smem);
    if (rc) return rc;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(p.n_cta);
        cfg.blockDim = dim3(THREADS);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = split_only ? 0 : 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, FDC_TC_KERNEL, p, tk, tv, nk, nv, split_only);
        if (e != cudaSuccess) return set_cuda_error(e);
    }
    note_launch();
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FDC_OK : set_cuda_error(e);
}

}  // namespace fdc
