// Integer kernels: Algorithm 1 (ready-set scheduling, Sec. 3.2) and Eq. 1 as row bitmaps
// (Sec. 3.3).  One warp per scene for the scheduler, one block per scene for the bitmaps.
#include "fdc_internal.h"

using namespace fdc;

#define FDC_CUDA(call)                                   \
    do {                                                 \
        cudaError_t e_ = (call);                         \
        if (e_ != cudaSuccess) return set_cuda_error(e_); \
    } while (0)

namespace {

__device__ __forceinline__ uint64_t warp_or64(uint64_t x)
{
    uint32_t lo = __reduce_or_sync(0xffffffffu, (uint32_t)x);
    uint32_t hi = __reduce_or_sync(0xffffffffu, (uint32_t)(x >> 32));
    return ((uint64_t)hi << 32) | lo;
}

// Algorithm 1 initialisation: d_v = indegree, S = {v : d_v = 0}.
__global__ void state_init_kernel(const PlanDev* __restrict__ plan, int batch, const int32_t* __restrict__ len,
                                  SceneState* __restrict__ state, int32_t* __restrict__ status)
{
    int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    if (s >= batch) return;
    const int n = plan->n;
    SceneState& st = state[s];
    uint64_t ready = 0;
    bool bad = false;
    for (int v = lane; v < FDC_MAX_NODES; v += 32) {
        int d = 0, tok = 0, lim = 0;
        if (v < n) {
            d = plan->indeg[v];
            tok = plan->nfixed[v];
            int c = plan->cap[v];
            lim = len ? len[(size_t)s * n + v] : c;
            if (lim < tok + 1) { lim = tok + 1; bad = true; }
            if (lim > c) { lim = c; bad = true; }
            if (d == 0) ready |= 1ull << v;
        }
        st.d[v] = d;
        st.tok[v] = tok;
        st.lim[v] = lim;
        st.node[v] = -1;
    }
    ready = warp_or64(ready);
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, FDC_DEV_LEN_RANGE);
    if (lane == 0) {
        st.ready = ready;
        st.done = 0;
        st.n_active = 0;
        st.pass = 0;
    }
}

// One iteration of Algorithm 1's loop for every scene: retire the fields that finished in
// the previous pass, lower d_u of their successors (d_u = unfinished parents, kept as a
// count and derived from the parent bitsets), admit fields with d_u = 0, emit the packed list.
__global__ void frontier_kernel(const PlanDev* __restrict__ plan, int batch, SceneState* __restrict__ state,
                                const uint8_t* __restrict__ finish, int32_t* __restrict__ n_active,
                                int32_t* __restrict__ node, int32_t* __restrict__ tok_idx,
                                int32_t* __restrict__ kv_row, int32_t* __restrict__ pos_id,
                                int32_t* __restrict__ all_done, int32_t* __restrict__ status,
                                int32_t* __restrict__ ticket)
{
    const int warps = blockDim.x >> 5;
    const int s = blockIdx.x * warps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int n = plan->n, maxa = plan->max_active, P = plan->P;
    int scene_live = 0;
    if (s < batch) {
        SceneState& st = state[s];
        uint64_t ready = st.ready, done = st.done;
        const int prev_a = st.n_active;
        // fields of the previous pass that are finished now
        uint64_t fin = 0;
        for (int b = lane; b < prev_a; b += 32) {
            int v = st.node[b];
            bool f = st.tok[v] >= st.lim[v];
            if (finish && finish[(size_t)s * maxa + b]) f = true;
            if (f) fin |= 1ull << v;
        }
        fin = warp_or64(fin);
        done |= fin;
        ready &= ~fin;
        // successors: d_u counts the unfinished parents (with multiplicity 1 per distinct parent
        // for readiness; the stored count keeps Alg. 1's meaning for inspection)
        uint64_t add = 0;
        for (int v = lane; v < n; v += 32) {
            uint64_t open = plan->par[v] & ~done;
            st.d[v] = __popcll(open);
            if (!((done >> v) & 1) && open == 0) add |= 1ull << v;
        }
        ready |= warp_or64(add);
        // packed list in ascending node id, at most max_active wide
        const int width = __popcll(ready);
        const int A = width < maxa ? width : maxa;
        __syncwarp();
        for (int v = lane; v < n; v += 32) {
            if ((ready >> v) & 1) {
                int b = __popcll(ready & ((1ull << v) - 1ull));
                if (b < maxa) {
                    int t = st.tok[v];
                    int row = P + plan->base[v] + t;
                    size_t o = (size_t)s * maxa + b;
                    node[o] = v;
                    tok_idx[o] = t;
                    kv_row[o] = row;
                    pos_id[o] = row;
                    st.node[b] = v;
                    st.tok[v] = t + 1;
                }
            }
        }
        for (int b = A + lane; b < maxa; b += 32) {
            size_t o = (size_t)s * maxa + b;
            node[o] = -1;
            tok_idx[o] = -1;
            kv_row[o] = -1;
            pos_id[o] = -1;
        }
        if (lane == 0) {
            st.ready = ready;
            st.done = done;
            st.n_active = A;
            st.pass += (A > 0);
            n_active[s] = A;
            if (width > maxa) atomicOr(status, FDC_DEV_FRONTIER_WIDE);
        }
        scene_live = ready != 0;
    }
    // all_done = no scene has a ready field: block OR, then last-block-done across the grid
    int block_live = __syncthreads_or(scene_live);
    if (threadIdx.x == 0) {
        if (block_live) atomicAdd(&ticket[1], 1);
        __threadfence();
        int t = atomicAdd(&ticket[0], 1);
        if (t == (int)gridDim.x - 1) {
            __threadfence();
            int live = atomicAdd(&ticket[1], 0);
            *all_done = live == 0;
            ticket[0] = 0;
            ticket[1] = 0;
        }
    }
}

// Eq. 1 as bitmaps: one block per scene.
__global__ void __launch_bounds__(256) build_masks_kernel(const PlanDev* __restrict__ plan, const SceneState* __restrict__ state,
                                                          uint64_t* __restrict__ mask, uint64_t* __restrict__ umask,
                                                          int32_t* __restrict__ tiles, int32_t* __restrict__ ntiles)
{
    extern __shared__ unsigned long long sm_umask[];   // [W]
    __shared__ int s_lo[FDC_MAX_NODES], s_tok[FDC_MAX_NODES], s_fix[FDC_MAX_NODES];
    __shared__ int s_warp_cnt[8];
    __shared__ int s_base_out;
    const int s = blockIdx.x;
    const int n = plan->n, W = plan->W, maxa = plan->max_active, P = plan->P, T = plan->T;
    const SceneState& st = state[s];
    const int A = st.n_active;
    for (int u = threadIdx.x; u < n; u += blockDim.x) {
        s_lo[u] = plan->base[u];
        s_tok[u] = st.tok[u];
        s_fix[u] = plan->nfixed[u];
    }
    for (int w = threadIdx.x; w < W; w += blockDim.x) sm_umask[w] = 0ull;
    __syncthreads();
    // per-branch words
    for (int i = threadIdx.x; i < maxa * W; i += blockDim.x) {
        const int b = i / W, w = i - b * W;
        uint64_t word = 0;
        if (b < A) {
            const int v = st.node[b];
            const uint64_t anc = plan->anc[v];
            const int w0 = w * 64;
            for (int u = 0; u < n; ++u) {
                // rows of field u this branch may see: all its real rows if u is an ancestor
                // (padding never), its own rows so far, else only u's fixed rows if they lie lower
                int vis = ((anc >> u) & 1) ? s_tok[u] : (u == v ? s_tok[u] : (u < v ? s_fix[u] : 0));
                int lo = s_lo[u] - w0, hi = lo + vis;
                if (lo < 0) lo = 0;
                if (hi > 64) hi = 64;
                if (hi > lo) {
                    uint64_t m = (hi - lo == 64) ? ~0ull : (((1ull << (hi - lo)) - 1ull) << lo);
                    word |= m;
                }
            }
            if (word) atomicOr(&sm_umask[w], (unsigned long long)word);
        }
        mask[((size_t)s * maxa + b) * W + w] = word;
    }
    __syncthreads();
    for (int w = threadIdx.x; w < W; w += blockDim.x) umask[(size_t)s * W + w] = sm_umask[w];
    // visited tiles, ascending (prefix tiles first by construction)
    const int ntile_max = plan->ntile_max;
    if (threadIdx.x == 0) s_base_out = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int t0 = 0; t0 < ntile_max; t0 += blockDim.x) {
        const int tile = t0 + threadIdx.x;
        bool vis = false;
        if (A > 0 && tile < ntile_max) {
            const int r0 = tile * FDC_TILE_ROWS;
            vis = r0 < P;
            if (!vis) vis = extract64((const uint64_t*)sm_umask, W, r0 - P) != 0ull;
            else if (r0 + FDC_TILE_ROWS > P) vis = true;
        }
        unsigned ball = __ballot_sync(0xffffffffu, vis);
        if (lane == 0) s_warp_cnt[warp] = __popc(ball);
        __syncthreads();
        int off = s_base_out;
        for (int wv = 0; wv < warp; ++wv) off += s_warp_cnt[wv];
        if (vis) tiles[(size_t)s * ntile_max + off + __popc(ball & ((1u << lane) - 1u))] = tile;
        __syncthreads();
        if (threadIdx.x == 0) {
            int tot = 0;
            for (int wv = 0; wv < (int)(blockDim.x >> 5); ++wv) tot += s_warp_cnt[wv];
            s_base_out += tot;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) ntiles[s] = s_base_out;
    (void)T;
}

// Algorithm 1's loop test, on the device: keeps a WHILE node of a CUDA graph going while some scene
// still has a ready field.
__global__ void loop_condition_kernel(const int32_t* __restrict__ all_done, int32_t* __restrict__ pass_count,
                                      int32_t max_passes, cudaGraphConditionalHandle handle, int32_t* __restrict__ status)
{
    const int32_t done_passes = *pass_count + 1;      // the pass whose tables were just replaced has been decoded
    *pass_count = done_passes;
    unsigned int more = *all_done == 0 ? 1u : 0u;
    if (more && done_passes >= max_passes) {           // never an endless loop, whatever the tables say
        more = 0u;
        atomicOr(status, FDC_DEV_LOOP_LIMIT);
    }
    cudaGraphSetConditional(handle, more);
}

}  // namespace

extern "C" {

int fdc_state_init(fdc_plan* p, int32_t batch, const int32_t* d_len, void* d_state, void* stream)
{
    if (!p || !d_state) return FDC_ERR_NULL;
    if (batch < 1 || batch > FDC_MAX_BATCH) return FDC_ERR_RANGE;
    {
        int rcf = flush_pending_append(p);
        if (rcf) return rcf;
    }
    const int warps = 4;
    ++p->tables_gen;                       // the pass tables change: work splits made from them are stale
    state_init_kernel<<<(batch + warps - 1) / warps, warps * 32, 0, (cudaStream_t)stream>>>(
        p->d, batch, d_len, (SceneState*)d_state, p->d_status);
    note_launch();
    FDC_CUDA(cudaGetLastError());
    return FDC_OK;
}

int fdc_frontier(fdc_plan* p, int32_t batch, void* d_state, const uint8_t* d_finish, int32_t* d_n_active,
                 int32_t* d_node, int32_t* d_tok_idx, int32_t* d_kv_row, int32_t* d_pos_id,
                 int32_t* d_all_done, void* stream)
{
    if (!p || !d_state || !d_n_active || !d_node || !d_tok_idx || !d_kv_row || !d_pos_id || !d_all_done)
        return FDC_ERR_NULL;
    if (batch < 1 || batch > FDC_MAX_BATCH) return FDC_ERR_RANGE;
    {
        int rcf = flush_pending_append(p);
        if (rcf) return rcf;
    }
    const int warps = batch < 8 ? batch : 8;
    ++p->tables_gen;                       // the pass tables change: work splits made from them are stale
    frontier_kernel<<<(batch + warps - 1) / warps, warps * 32, 0, (cudaStream_t)stream>>>(
        p->d, batch, (SceneState*)d_state, d_finish, d_n_active, d_node, d_tok_idx, d_kv_row, d_pos_id,
        d_all_done, p->d_status, p->d_ticket);
    note_launch();
    FDC_CUDA(cudaGetLastError());
    return FDC_OK;
}

int fdc_build_masks(fdc_plan* p, int32_t batch, const void* d_state, uint64_t* d_mask, uint64_t* d_umask,
                    int32_t* d_tiles, int32_t* d_ntiles, void* stream)
{
    if (!p || !d_state || !d_mask || !d_umask || !d_tiles || !d_ntiles) return FDC_ERR_NULL;
    if (batch < 1 || batch > FDC_MAX_BATCH) return FDC_ERR_RANGE;
    {
        int rcf = flush_pending_append(p);
        if (rcf) return rcf;
    }
    ++p->tables_gen;                       // the pass tables change: work splits made from them are stale
    build_masks_kernel<<<batch, 256, p->h.W * sizeof(uint64_t), (cudaStream_t)stream>>>(
        p->d, (const SceneState*)d_state, d_mask, d_umask, d_tiles, d_ntiles);
    note_launch();
    FDC_CUDA(cudaGetLastError());
    return FDC_OK;
}

int fdc_loop_condition(fdc_plan* p, const int32_t* d_all_done, int32_t* d_pass_count, int32_t max_passes,
                       unsigned long long cond_handle, void* stream)
{
    if (!p || !d_all_done || !d_pass_count) return FDC_ERR_NULL;
    if (max_passes < 1) return FDC_ERR_RANGE;
    {
        int rcf = flush_pending_append(p);
        if (rcf) return rcf;
    }
    loop_condition_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(d_all_done, d_pass_count, max_passes,
                                                             (cudaGraphConditionalHandle)cond_handle, p->d_status);
    note_launch();
    FDC_CUDA(cudaGetLastError());
    return FDC_OK;
}

}  // extern "C"
