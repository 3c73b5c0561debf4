// Internal declarations shared by the translation units of libfdc (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fdc.h"

#define FDC_PAIR_COUNTERS 65536
// Work split of the tcgen05 attention kernel: the layers of one forward pass see the same
// per-scene counts, so the split is computed once per pass (by a launch of the kernel that does
// nothing else, before the pass's first attention launch) and kept here with the counts it was
// computed from; the attention launches only check that the counts are unchanged.  Layout, in
// int32: [0..15] header, [16..) n_active[FDC_MEMO_BATCH], tiles[FDC_MEMO_BATCH],
// prev[FDC_MEMO_BATCH + 1], [FDC_MEMO_ENTRIES..) first and last unit of each CTA (2 x int64).
#define FDC_MEMO_BATCH 256
#define FDC_MEMO_CTAS 256
#define FDC_MEMO_ENTRIES 800
#define FDC_MEMO_INTS (FDC_MEMO_ENTRIES + 4 * FDC_MEMO_CTAS)

namespace fdc {

// Device-resident template tables (built on the host by fdc_plan_graph).
struct PlanDev {
    int32_t  n, m, P, T, W, max_active, ntile_max, pad0;
    uint64_t anc[FDC_MAX_NODES];     // bit u of anc[v]: a path u -> ... -> v exists (Eq. 1)
    uint64_t par[FDC_MAX_NODES];     // bit u of par[v]: edge (u, v)
    int32_t  base[FDC_MAX_NODES + 1];
    int32_t  pad1;
    int32_t  cap[FDC_MAX_NODES];
    int32_t  nfixed[FDC_MAX_NODES];
    int32_t  indeg[FDC_MAX_NODES];   // incoming edges, duplicates counted (Alg. 1's initial d_v)
};

// Per-scene scheduler state (caller-owned device memory, opaque to the caller).
struct alignas(16) SceneState {
    uint64_t ready;                  // S of Algorithm 1 as a node bitset
    uint64_t done;                   // finished fields
    int32_t  n_active;               // width of the last emitted pass
    int32_t  pass;                   // passes emitted so far
    int32_t  pad[2];
    int32_t  d[FDC_MAX_NODES];       // unfinished prerequisites of each field
    int32_t  tok[FDC_MAX_NODES];     // rows of the field present in the cache (after this pass's append)
    int32_t  lim[FDC_MAX_NODES];     // the field is finished when tok reaches lim
    int32_t  node[FDC_MAX_NODES];    // packed list of the last emitted pass
};

}  // namespace fdc

// Arguments of an fdc_kv_append call that has been recorded instead of launched (fused append).
struct fdc_pending_append {
    int            valid;
    fdc_kv_desc    kv;
    int32_t        layer;
    const int32_t* d_n_active;
    const int32_t* d_kv_row;
    const void*    d_k_new;
    const void*    d_v_new;
    void*          stream;
};

// Everything the work split of the tcgen05 attention kernel depends on (host side).
struct fdc_split_key {
    uint32_t       tables_gen;
    const int32_t* d_n_active;
    const int32_t* d_ntiles;
    int32_t        batch, hkv, n_cta, P;
    void*          stream;
    int            valid;
};

struct fdc_plan {
    fdc::PlanDev  h;                 // host copy
    fdc::PlanDev* d;                 // device copy
    int32_t*      d_status;          // sticky FDC_DEV_* bits
    int32_t*      d_ticket;          // [2] scratch of the frontier kernel's cross-block reduction
    int32_t*      d_pair_cnt;        // [FDC_PAIR_COUNTERS] arrivals per (scene, KV head) of the fused combine (zero between calls)
    int32_t*      d_split_memo;      // [FDC_MEMO_INTS] work split of the current pass and the counts it was made from
    uint32_t      tables_gen;        // bumped by every call that rewrites the pass tables (state_init, frontier, build_masks)
    uint32_t      split_gen;         // number of the last split launch (stored in the memo's header)
    fdc_split_key split_key;         // what the memo was computed for
    uint32_t      attn_gen;          // tables_gen at the last attention launch of the tcgen05 kernel
    void*         attn_stream;       // and its stream
    int           attn_gen_valid;
    int           fuse_append;       // fdc_set_fused_append
    fdc_pending_append pend;         // recorded append waiting for its attention call
    int           device;
    int           sm_count;
    int           attn_kernel;       // 0 auto
    void*         prof;              // event records of fdc_profile (nullptr when never enabled)
    int           prof_on;
    int32_t*      succ_ptr;          // host CSR successor lists (kept for inspection)
    int32_t*      succ;
};

namespace fdc {

// Attention launch parameters (passed by value).
struct AttnParams {
    const void*     k;               // layer base
    const void*     v;
    int64_t         stride_scene, stride_head, stride_row;   // elements
    const void*     q;               // [batch][max_active][hq][D]
    void*           out;
    const uint64_t* mask;            // [batch][max_active][W]
    const int32_t*  tiles;           // [batch][ntile_max]
    const int32_t*  ntiles;          // [batch]
    const int32_t*  n_active;        // [batch]
    float*          ws_o;            // [slots][mmax][D]
    float*          ws_ml;           // [slots][mmax][2]
    int32_t         batch, hkv, hq, group, max_active, mmax, W, P, rows, ntile_max, n_cta;
    float           scale_log2;      // softmax scale * log2(e)
    int32_t*        status;          // sticky FDC_DEV_* bits
    int32_t*        pair_cnt;        // per (scene, KV head) arrival counters: the split kernel also combines (nullptr: it does not)
    int32_t*        split_memo;      // [FDC_MEMO_INTS] (nullptr: the work split is always computed)
    uint32_t        seq;             // number of the split launch the memo must come from
    int32_t         early;           // the pass tables, the memo and the prefix rows were complete before the kernel
                                     // preceding this one in the stream began: they may be read ahead of the dependency wait
    const int32_t*  app_row;         // fused append: [batch][max_active] cache row of each branch's new K/V vector (nullptr: none)
    const void*     app_k;           // [batch][max_active][hkv][D]
    const void*     app_v;
};

extern int64_t g_launches;
void note_launch();
int  set_cuda_error(cudaError_t e);                  // records the message, returns FDC_ERR_CUDA

int launch_attn_ref(const AttnParams& p, int dtype, int head_dim, cudaStream_t st);
int launch_attn_mma(const AttnParams& p, int head_dim, cudaStream_t st);
int launch_attn_tc(const AttnParams& p, int head_dim, cudaStream_t st);
int launch_attn_tc_split(const AttnParams& p, int head_dim, cudaStream_t st);   // computes the work split only (into p.split_memo)
int launch_attn_combine(const AttnParams& p, int dtype, int head_dim, cudaStream_t st);
void prof_destroy(fdc_plan* plan);
int  check_kv_desc(const fdc_plan* plan, const fdc_kv_desc* kv, int32_t layer);
bool takes_tc_kernel(const fdc_plan* plan, const fdc_kv_desc* kv);   // fdc_decode_attn would run the tcgen05 kernel with the combine fused in
int  launch_kv_append(fdc_plan* plan, const fdc_kv_desc* kv, int32_t layer, const int32_t* d_n_active, const int32_t* d_kv_row,
                      const void* d_k_new, const void* d_v_new, void* stream);
int  flush_pending_append(fdc_plan* plan);     // launches a recorded append on its own (no-op when there is none)

// cudaFuncAttributeMaxDynamicSharedMemorySize is kept by the runtime per device: `set` remembers,
// per device ordinal, what this process has already asked for on behalf of one kernel.
constexpr int kMaxDevices = 64;
inline int raise_dynamic_smem(const void* kernel, size_t bytes, size_t (&set)[kMaxDevices])
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_cuda_error(e);
    const bool known = dev >= 0 && dev < kMaxDevices;
    if (known && bytes <= set[dev]) return FDC_OK;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return set_cuda_error(e);
    if (known) set[dev] = bytes;
    return FDC_OK;
}

// ----------------------------------------------------------------------------------
// device helpers
// ----------------------------------------------------------------------------------
#ifdef __CUDACC__
// 64 bits of a bitmap of `W` words starting at bit position `start` (may be negative or run
// past the end: bits outside [0, 64*W) read as 0).
__device__ __forceinline__ uint64_t extract64(const uint64_t* __restrict__ words, int W, int start)
{
    if (start <= -64) return 0ull;
    if (start < 0) return W > 0 ? (words[0] << (-start)) : 0ull;
    int w = start >> 6, sh = start & 63;
    if (w >= W) return 0ull;
    uint64_t lo = words[w] >> sh;
    if (sh && w + 1 < W) lo |= words[w + 1] << (64 - sh);
    return lo;
}

// Visibility of the 64 rows of KV tile `tile` for one branch: prefix rows are all visible.
__device__ __forceinline__ uint64_t tile_rowmask(const uint64_t* __restrict__ words, int W, int P, int tile)
{
    int r0 = tile * FDC_TILE_ROWS;
    int npre = P - r0;
    uint64_t pm = npre >= 64 ? ~0ull : (npre <= 0 ? 0ull : ((1ull << npre) - 1ull));
    if (npre >= 64) return pm;
    return pm | extract64(words, W, r0 - P);
}

// Work split shared by the split pass and the combine pass: unit u (one KV tile of one
// (scene, KV head) pair, pairs in scene-major order) belongs to CTA floor(u * n_cta / U).
__device__ __forceinline__ long long cta_first_unit(long long c, long long U, long long n_cta)
{
    return (c * U + n_cta - 1) / n_cta;
}
__device__ __forceinline__ int unit_cta(long long u, long long U, long long n_cta)
{
    return (int)((u * n_cta) / U);
}
#endif

}  // namespace fdc
