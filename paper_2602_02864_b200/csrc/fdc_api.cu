// Host side of the C ABI: template planning (Sec. 3.2, Eq. 1), size queries, status.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "fdc_internal.h"

namespace fdc {

static std::atomic<int64_t> g_launch_counter{0};
static thread_local char g_cuda_msg[256] = "";

void note_launch() { g_launch_counter.fetch_add(1, std::memory_order_relaxed); }

int set_cuda_error(cudaError_t e)
{
    snprintf(g_cuda_msg, sizeof(g_cuda_msg), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return FDC_ERR_CUDA;
}

}  // namespace fdc

using namespace fdc;

#define FDC_CUDA(call)                                   \
    do {                                                 \
        cudaError_t e_ = (call);                         \
        if (e_ != cudaSuccess) return set_cuda_error(e_); \
    } while (0)

extern "C" {

int64_t fdc_launch_count(void) { return g_launch_counter.load(); }

const char* fdc_last_cuda_error(void) { return g_cuda_msg; }

const char* fdc_strerror(int code)
{
    switch (code) {
        case FDC_OK: return "ok";
        case FDC_ERR_NULL: return "null pointer";
        case FDC_ERR_CYCLE: return "dependency graph has a cycle";
        case FDC_ERR_RANGE: return "argument out of range";
        case FDC_ERR_SHAPE: return "unsupported shape or stride";
        case FDC_ERR_DTYPE: return "unsupported dtype";
        case FDC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case FDC_ERR_CUDA: return "CUDA runtime error";
        case FDC_ERR_DEVICE: return "device recorded an anomaly";
        case FDC_ERR_STATIC_LIMIT: return "problem needs more scratch than the built-in static buffer (FDC_STATIC_WS_BYTES)";
        default: return "unknown error";
    }
}

int fdc_plan_graph(const fdc_graph_desc* g, fdc_plan** out)
{
    if (!g || !out) return FDC_ERR_NULL;
    *out = nullptr;
    const int n = g->n_nodes, m = g->n_edges;
    if (n < 1 || n > FDC_MAX_NODES || m < 0) return FDC_ERR_RANGE;
    if (!g->slot_cap || (m > 0 && !g->edges)) return FDC_ERR_NULL;
    if (g->prefix_len < 0 || g->max_active < 1 || g->max_active > FDC_MAX_NODES) return FDC_ERR_RANGE;

    PlanDev h;
    memset(&h, 0, sizeof(h));
    h.n = n;
    h.m = m;
    h.P = g->prefix_len;
    h.max_active = g->max_active;
    long long T = 0;
    for (int v = 0; v < n; ++v) {
        int c = g->slot_cap[v];
        int f = g->n_fixed ? g->n_fixed[v] : 0;
        if (c < 1 || f < 0 || f >= c) return FDC_ERR_RANGE;
        h.base[v] = (int32_t)T;
        h.cap[v] = c;
        h.nfixed[v] = f;
        T += c;
        if (T + h.P > (1ll << 30)) return FDC_ERR_RANGE;
    }
    h.base[n] = (int32_t)T;
    h.T = (int32_t)T;
    h.W = (int32_t)((T + 63) / 64);
    h.ntile_max = (int32_t)((h.P + T + FDC_TILE_ROWS - 1) / FDC_TILE_ROWS);

    for (int e = 0; e < m; ++e) {
        int a = g->edges[2 * e], b = g->edges[2 * e + 1];
        if (a < 0 || a >= n || b < 0 || b >= n) return FDC_ERR_RANGE;
        if (a == b) return FDC_ERR_CYCLE;
        h.par[b] |= 1ull << a;
        h.indeg[b] += 1;
    }
    // Topological peeling on parent bitsets (Kahn): a node is peeled once all its parents
    // are; its ancestor set is the union of its parents and their ancestor sets.  Nodes
    // that can never be peeled lie on (or behind) a cycle.
    uint64_t peeled = 0;
    const uint64_t all = n == 64 ? ~0ull : ((1ull << n) - 1ull);
    for (int round = 0; round < n && peeled != all; ++round) {
        uint64_t now = 0;
        for (int v = 0; v < n; ++v)
            if (!((peeled >> v) & 1) && (h.par[v] & ~peeled) == 0) now |= 1ull << v;
        if (!now) return FDC_ERR_CYCLE;
        for (int v = 0; v < n; ++v) {
            if (!((now >> v) & 1)) continue;
            uint64_t a = h.par[v];
            for (int u = 0; u < n; ++u)
                if ((h.par[v] >> u) & 1) a |= h.anc[u];
            h.anc[v] = a;
        }
        peeled |= now;
    }
    if (peeled != all) return FDC_ERR_CYCLE;

    fdc_plan* p = new (std::nothrow) fdc_plan;
    if (!p) return FDC_ERR_CUDA;
    memset(p, 0, sizeof(*p));
    p->h = h;
    p->succ_ptr = (int32_t*)calloc(n + 1, sizeof(int32_t));
    p->succ = (int32_t*)calloc(m > 0 ? m : 1, sizeof(int32_t));
    for (int e = 0; e < m; ++e) p->succ_ptr[g->edges[2 * e] + 1]++;
    for (int v = 0; v < n; ++v) p->succ_ptr[v + 1] += p->succ_ptr[v];
    {
        std::vector<int32_t> fill(p->succ_ptr, p->succ_ptr + n);
        for (int e = 0; e < m; ++e) p->succ[fill[g->edges[2 * e]]++] = g->edges[2 * e + 1];
    }
    cudaError_t e = cudaGetDevice(&p->device);
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, p->device);
    if (e == cudaSuccess) {
        p->sm_count = prop.multiProcessorCount;
        e = cudaMalloc((void**)&p->d, sizeof(PlanDev));
    }
    if (e == cudaSuccess) e = cudaMalloc((void**)&p->d_status, (4 + FDC_PAIR_COUNTERS + FDC_MEMO_INTS) * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemcpy(p->d, &p->h, sizeof(PlanDev), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(p->d_status, 0, (4 + FDC_PAIR_COUNTERS + FDC_MEMO_INTS) * sizeof(int32_t));
    if (e != cudaSuccess) {
        int rc = set_cuda_error(e);
        fdc_plan_destroy(p);
        return rc;
    }
    p->d_ticket = p->d_status + 2;
    p->d_pair_cnt = p->d_status + 4;
    p->d_split_memo = p->d_pair_cnt + FDC_PAIR_COUNTERS;
    p->fuse_append = 0;
    p->pend.valid = 0;
    *out = p;
    return FDC_OK;
}

int fdc_plan_destroy(fdc_plan* p)
{
    if (!p) return FDC_ERR_NULL;
    flush_pending_append(p);              // a recorded append is still owed to the cache
    prof_destroy(p);
    if (p->d) cudaFree(p->d);
    if (p->d_status) cudaFree(p->d_status);
    free(p->succ_ptr);
    free(p->succ);
    delete p;
    return FDC_OK;
}

int fdc_plan_query(const fdc_plan* p, int32_t batch, fdc_sizes* out)
{
    if (!p || !out) return FDC_ERR_NULL;
    if (batch < 1 || batch > FDC_MAX_BATCH) return FDC_ERR_RANGE;
    out->cot_rows = p->h.T;
    out->mask_words = p->h.W;
    out->ntile_max = p->h.ntile_max;
    out->max_active = p->h.max_active;
    out->state_bytes = (size_t)batch * sizeof(SceneState);
    out->mask_bytes = (size_t)batch * p->h.max_active * p->h.W * sizeof(uint64_t);
    out->umask_bytes = (size_t)batch * p->h.W * sizeof(uint64_t);
    out->tiles_bytes = (size_t)batch * p->h.ntile_max * sizeof(int32_t);
    return FDC_OK;
}

int fdc_plan_tables(const fdc_plan* p, uint64_t* anc, uint64_t* par, int32_t* base, int32_t* indegree)
{
    if (!p) return FDC_ERR_NULL;
    const int n = p->h.n;
    if (anc) memcpy(anc, p->h.anc, n * sizeof(uint64_t));
    if (par) memcpy(par, p->h.par, n * sizeof(uint64_t));
    if (base) memcpy(base, p->h.base, (n + 1) * sizeof(int32_t));
    if (indegree) memcpy(indegree, p->h.indeg, n * sizeof(int32_t));
    return FDC_OK;
}

int fdc_plan_critical_path(const fdc_plan* p, const int32_t* len, int32_t* steps, int32_t* finish)
{
    if (!p || !len || !steps) return FDC_ERR_NULL;
    const int n = p->h.n;
    int32_t fin[FDC_MAX_NODES];
    for (int v = 0; v < n; ++v) {
        if (len[v] < p->h.nfixed[v] + 1 || len[v] > p->h.cap[v]) return FDC_ERR_RANGE;
        fin[v] = -1;
    }
    // relax in dependency order: a node is settled once all its parents are
    int settled = 0, best = 0;
    while (settled < n) {
        for (int v = 0; v < n; ++v) {
            if (fin[v] >= 0) continue;
            int32_t start = 0;
            bool ok = true;
            for (int u = 0; u < n && ok; ++u)
                if ((p->h.par[v] >> u) & 1) {
                    if (fin[u] < 0) ok = false;
                    else if (fin[u] > start) start = fin[u];
                }
            if (!ok) continue;
            fin[v] = start + (len[v] - p->h.nfixed[v]);
            if (fin[v] > best) best = fin[v];
            ++settled;
        }
    }
    *steps = best;
    if (finish) memcpy(finish, fin, n * sizeof(int32_t));
    return FDC_OK;
}

int fdc_status(fdc_plan* p, int32_t* host_bits, int32_t clear, void* stream)
{
    if (!p || !host_bits) return FDC_ERR_NULL;
    {
        int rcf = flush_pending_append(p);
        if (rcf) return rcf;
    }
    cudaStream_t st = (cudaStream_t)stream;
    FDC_CUDA(cudaMemcpyAsync(host_bits, p->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    if (clear) {
        // a launch that gave up may have left arrival counters of the fused combine behind
        FDC_CUDA(cudaMemsetAsync(p->d_status, 0, sizeof(int32_t), st));
        FDC_CUDA(cudaMemsetAsync(p->d_pair_cnt, 0, FDC_PAIR_COUNTERS * sizeof(int32_t), st));
    }
    FDC_CUDA(cudaStreamSynchronize(st));
    return *host_bits ? FDC_ERR_DEVICE : FDC_OK;
}

}  // extern "C"
