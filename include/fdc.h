/* fdc.h - C ABI of the dependency-masked multi-branch decode path (B200, sm_100a).
 *
 * The method (FastDriveCoT): a chain-of-thought template is a DAG of fields; every field
 * whose prerequisites are complete decodes one token in the same forward pass
 * (Algorithm 1, Sec. 3.2).  All parallel fields are packed into ONE sequence sharing one KV
 * cache; an attention mask derived from the graph lets a token attend a field iff that
 * field is an ancestor of its own (Eq. 1, Sec. 3.3), fixed-length slots make every position
 * id known in advance, and padding is visible to nobody and never processed (Sec. 3.3).
 *
 * One forward pass through this library, everything stream-ordered on the device:
 *     fdc_frontier      Algorithm 1 body: retire finished fields, admit newly ready ones,
 *                       emit this pass's packed branch list (node, token, KV row, position)
 *     fdc_build_masks   Eq. 1 as per-branch row bitmaps + the list of KV tiles anyone sees
 *     per layer:
 *       fdc_kv_append   write each branch's new K/V vector at its slot row
 *       fdc_decode_attn masked attention of all branches x all GQA heads of a scene over the
 *                       shared cache, reading each visible KV row once (Sec. 3.3, "Reduced
 *                       Memory Bottleneck"), split over the GPU and combined
 *
 * Conventions
 *   - Every function returns FDC_OK (0) or a negative FDC_ERR_*; nothing throws, aborts or
 *     traps.  Host-side argument errors are reported before anything is launched.
 *   - "host" pointers are dereferenced by the calling thread; "device" pointers are only
 *     handed to kernels.  All device buffers are CALLER-OWNED (sizes from fdc_plan_query /
 *     fdc_attn_workspace_bytes); the library owns only the opaque fdc_plan.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  fdc_state_init,
 *     fdc_frontier, fdc_build_masks, fdc_kv_append and fdc_decode_attn only enqueue work;
 *     they never synchronise or read device memory on the host.
 *   - Device-side anomalies (a KV row outside the cache, a frontier wider than max_active,
 *     a field length outside its slot) never fault: the offending item is clamped or
 *     skipped and a sticky bit is set in the plan's status word (fdc_status).
 *   - A plan is bound to the CUDA device that was current in fdc_plan_graph.
 */
#ifndef FDC_H_
#define FDC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FDC_MAX_NODES   64   /* fields per template (one 64-bit word per node set)          */
#define FDC_TILE_ROWS   64   /* KV rows per tile of the visited-tile list                   */
#define FDC_MAX_QROWS   128  /* max_active * (hq / hkv): query rows served by one KV read   */
#define FDC_MAX_BATCH   4096 /* scenes per call                                             */
#define FDC_STATIC_WS_BYTES (16u << 20) /* built-in scratch of fdc_decode_attn_static, per GPU  */

enum {
    FDC_OK            =  0,
    FDC_ERR_NULL      = -1,  /* a required pointer is NULL                                  */
    FDC_ERR_CYCLE     = -2,  /* the dependency graph has a directed cycle or a self loop    */
    FDC_ERR_RANGE     = -3,  /* node id, node count, slot, n_fixed, max_active, layer, batch out of range */
    FDC_ERR_SHAPE     = -4,  /* hq % hkv, head_dim not in {64,128}, rows < P+T, too many query rows, strides */
    FDC_ERR_DTYPE     = -5,  /* dtype is neither FDC_F32 nor FDC_BF16                       */
    FDC_ERR_WORKSPACE = -6,  /* workspace missing, misaligned or smaller than required      */
    FDC_ERR_CUDA      = -7,  /* a CUDA runtime call failed (see fdc_last_cuda_error)        */
    FDC_ERR_DEVICE    = -8,  /* fdc_status: the device recorded an anomaly                  */
    FDC_ERR_STATIC_LIMIT = -9 /* fdc_decode_attn_static: the problem needs more scratch than */
                             /* FDC_STATIC_WS_BYTES; nothing was launched                   */
};

enum { FDC_F32 = 0, FDC_BF16 = 1 };

/* bits of the sticky device status word */
enum {
    FDC_DEV_ROW_RANGE     = 1,  /* fdc_kv_append: kv_row outside [0, rows): row skipped      */
    FDC_DEV_FRONTIER_WIDE = 2,  /* fdc_frontier: more ready fields than max_active: clamped, */
                                /* the others wait for a later pass                          */
    FDC_DEV_LEN_RANGE     = 4,  /* fdc_state_init: a length outside [n_fixed+1, C]: clamped  */
    FDC_DEV_TIMEOUT       = 8,  /* fdc_decode_attn: a bounded in-kernel wait ran out; the    */
                                /* launch's output is invalid                                */
    FDC_DEV_SCORE_RANGE   = 16, /* fdc_decode_attn: a score rose more than 2^100 above its   */
                                /* softmax reference within three rounds (128 KV rows each)  */
                                /* of a reference update: the output may have overflowed     */
    FDC_DEV_TILE_LIST     = 32, /* fdc_decode_attn: d_tiles does not list the whole prefix   */
                                /* tiles first, as entries 0, 1, 2, ... (fdc_build_masks     */
                                /* always does); rows nobody may see could have been read    */
    FDC_DEV_LOOP_LIMIT    = 64  /* fdc_loop_condition: max_passes reached with fields still  */
                                /* ready: the device loop was stopped                        */
};

typedef struct fdc_plan fdc_plan;

/* Template description (Sec. 3.1-3.2).  All pointers are HOST memory, read during the call. */
typedef struct {
    int32_t        n_nodes;     /* fields, 1..FDC_MAX_NODES; node id = template order        */
    int32_t        n_edges;
    const int32_t* edges;       /* [n_edges][2] = (src, dst): dst needs src complete          */
    const int32_t* slot_cap;    /* [n_nodes] C[v] >= 1: rows reserved for field v (Sec. 3.3) */
    const int32_t* n_fixed;     /* [n_nodes] pre-filled field-name rows at the head of each  */
                                /* slot (0 <= n_fixed < C), or NULL for none                  */
    int32_t        prefix_len;  /* P >= 0: shared vision+prompt rows, visible to everyone    */
    int32_t        max_active;  /* branch slots per scene per pass, 1..FDC_MAX_NODES         */
} fdc_graph_desc;

/* KV cache view.  k and v are DEVICE pointers to element [scene 0][layer 0][head 0][row 0][0];
 * strides are in ELEMENTS; head_dim elements of a row are contiguous.  Row r of a scene is
 * the prefix for r < P and template row r - P otherwise.  Required: every stride a multiple
 * of 8 elements and k, v 16-byte aligned (128-bit accesses). */
typedef struct {
    void*   k;
    void*   v;
    int32_t dtype;              /* FDC_F32 | FDC_BF16 (also the dtype of q, k_new, v_new, out) */
    int32_t batch, layers, hkv, hq, head_dim, rows;
    int64_t stride_scene, stride_layer, stride_head, stride_row;
} fdc_kv_desc;

/* Sizes of the caller-owned buffers for `batch` scenes. */
typedef struct {
    int32_t cot_rows;           /* T = sum of C[v]                                            */
    int32_t mask_words;         /* W = ceil(T / 64) words per branch bitmap                   */
    int32_t ntile_max;          /* entries per scene of the tile list = ceil((P+T)/64)        */
    int32_t max_active;
    size_t  state_bytes;        /* d_state                                                    */
    size_t  mask_bytes;         /* d_mask  : uint64 [batch][max_active][W]                    */
    size_t  umask_bytes;        /* d_umask : uint64 [batch][W]                                */
    size_t  tiles_bytes;        /* d_tiles : int32  [batch][ntile_max]                        */
} fdc_sizes;

/* Sec. 3.2 (the dependency graph) and Eq. 1.  Validates the template (ids in range, no
 * cycle), builds on the host the parent sets, successor lists, the ANCESTOR set of every
 * node (transitive closure of E: bit u of anc[v] <=> a path u -> ... -> v) and the slot
 * bases base[v] = sum_{u<v} C[u], and copies them to the current device.  Host call;
 * allocates the plan (a few KB of device memory); synchronises.  *out is set on success. */
int fdc_plan_graph(const fdc_graph_desc* desc, fdc_plan** out);
int fdc_plan_destroy(fdc_plan* plan);

int fdc_plan_query(const fdc_plan* plan, int32_t batch, fdc_sizes* out);

/* Host copies of the plan's tables, for inspection and tests: anc/par uint64 [n],
 * base int32 [n+1], indegree int32 [n].  Any output pointer may be NULL. */
int fdc_plan_tables(const fdc_plan* plan, uint64_t* anc, uint64_t* par, int32_t* base, int32_t* indegree);

/* Sec. 3.2: the minimum number of forward passes = the largest cumulative number of
 * generated tokens along any dependency chain.  len is HOST int32 [n] (rows of each field
 * including its fixed ones); finish (HOST int32 [n], may be NULL) receives the 1-based pass in
 * which each field emits its last token.  Host-only arithmetic. */
int fdc_plan_critical_path(const fdc_plan* plan, const int32_t* len, int32_t* steps, int32_t* finish);

/* Algorithm 1 initialisation for `batch` scenes: d_v = indegree, S = sources, no field has
 * generated anything (tok[v] = n_fixed[v]).  d_len: DEVICE int32 [batch][n] = the number of
 * rows after which field v of scene s is finished when no finish flag arrives earlier
 * (synthetic runs: the field's true length), or NULL to use the slot C[v] (truncation to the
 * fixed length, Sec. 3.3).  Values are clamped to [n_fixed+1, C]. */
int fdc_state_init(fdc_plan* plan, int32_t batch, const int32_t* d_len, void* d_state, void* stream);

/* Algorithm 1, one loop iteration (Sec. 3.2).  First retires the fields of the previous pass
 * that finished - branch slot b of scene s is finished if d_finish[s][b] != 0 (DEVICE uint8
 * [batch][max_active], e.g. "end of field sampled"; may be NULL) or its row count reached its
 * limit - lowers d_u of their successors and admits those that reach 0.  Then emits the packed
 * list of this pass, one entry per ready field in ascending node id:
 *   d_n_active int32 [batch]               A = ready fields (<= max_active)
 *   d_node     int32 [batch][max_active]   field id, -1 in unused slots
 *   d_tok_idx  int32 [batch][max_active]   t: index within the slot of the token decoded now
 *   d_kv_row   int32 [batch][max_active]   P + base[v] + t (Sec. 3.3: fixed slots), -1 unused
 *   d_pos_id   int32 [batch][max_active]   the same value: position id = reserved row
 *   d_all_done int32 [1]                   1 iff no scene has a ready field left
 * A field admitted in this call decodes its first token in this pass; a field that finishes
 * in this pass is retired by the NEXT call.  All outputs are DEVICE memory. */
int fdc_frontier(fdc_plan* plan, int32_t batch, void* d_state, const uint8_t* d_finish,
                 int32_t* d_n_active, int32_t* d_node, int32_t* d_tok_idx, int32_t* d_kv_row,
                 int32_t* d_pos_id, int32_t* d_all_done, void* stream);

/* Eq. 1 + Sec. 3.3 as bitmaps, for the pass fdc_frontier just emitted (reads d_state).
 *   d_mask  uint64 [batch][max_active][W]  bit i of word w <=> template row 64w+i is visible
 *           to that branch: a real (non-padding) row of an ancestor field, a row <= t of its
 *           own field, or a fixed field-name row at a lower position.  Unused slots: 0.
 *           Prefix rows are not in the bitmap: they are visible to every branch.
 *   d_umask uint64 [batch][W]              OR over the scene's branches
 *   d_tiles int32  [batch][ntile_max], d_ntiles int32 [batch]
 *           ascending ids of the KV tiles (rows 64i..64i+63 of the scene's cache, prefix
 *           included) holding at least one row visible to some branch; 0 tiles for a scene
 *           with no active branch. */
int fdc_build_masks(fdc_plan* plan, int32_t batch, const void* d_state, uint64_t* d_mask,
                    uint64_t* d_umask, int32_t* d_tiles, int32_t* d_ntiles, void* stream);

/* Sec. 3.3 (shared KV cache, reused by all later passes): for every scene s and branch
 * b < d_n_active[s], copy d_k_new/d_v_new [batch][max_active][hkv][head_dim] into cache row
 * d_kv_row[s][b] of `layer`.  Padding rows are never written.  Rows outside [0, rows) are
 * skipped and flagged in the plan's status word.  d_k_new, d_v_new and d_kv_row are read for
 * every branch slot, idle ones included (the loads are issued before d_n_active is known), so
 * all of [batch][max_active] must be addressable; what idle slots hold does not matter. */
int fdc_kv_append(fdc_plan* plan, const fdc_kv_desc* kv, int32_t layer, const int32_t* d_n_active,
                  const int32_t* d_kv_row, const void* d_k_new, const void* d_v_new, void* stream);

/* Sec. 3.1 / Fig. 3: every line of the template starts with its field name, whose tokens are known
 * in advance and "pre-filled".  Writes the K/V of those rows of `layer` for every scene, once, at
 * prefill time: d_k_fixed / d_v_fixed are DEVICE [batch][hkv][F][head_dim] in the cache dtype,
 * F = sum of n_fixed[v], rows ordered by field (template order) and then by token; row j of field v
 * goes to cache row P + base[v] + j.  Nothing is launched for a template without fixed rows.  Rows
 * outside [0, rows) are skipped and flagged (FDC_DEV_ROW_RANGE). */
int fdc_kv_write_fixed(fdc_plan* plan, const fdc_kv_desc* kv, int32_t layer, const void* d_k_fixed,
                       const void* d_v_fixed, void* stream);

/* Scratch for fdc_decode_attn (split partials); depends on the plan, the cache shape and the
 * device's SM count. */
int fdc_attn_workspace_bytes(const fdc_plan* plan, const fdc_kv_desc* kv, size_t* bytes);

/* The masked attention of one layer for the pass described by d_n_active/d_mask/d_tiles
 * (Sec. 3.3): for scene s, branch b < A, query head h (KV head h / (hq/hkv)),
 *     out = softmax_r(scale * q . K[r]) V[r]   over the rows r visible to branch b
 * (prefix rows and the rows set in d_mask[s][b]).  q and out: DEVICE [batch][max_active][hq]
 * [head_dim] in the cache dtype; rows of unused branch slots are not touched.  Scores,
 * softmax and accumulation are fp32; bf16 output is rounded to nearest even.  Each visited
 * KV tile is read once for all branches and all heads of its KV group; invisible K/V rows
 * may hold anything (NaN included).  d_tiles must be what fdc_build_masks wrote: ascending,
 * the whole tiles of the prefix first (entry j = tile j); the kernel decides by list position
 * which tiles can hold rows that nobody may see (FDC_DEV_TILE_LIST if the list disagrees).
 * d_workspace: DEVICE, 256-byte aligned,
 * >= fdc_attn_workspace_bytes; its contents are undefined afterwards.
 * The tcgen05 kernel merges its split partials itself and keeps per-(scene, KV head) arrival
 * counters in the plan.  Its work split depends only on d_n_active / d_ntiles, so it is computed once
 * per pass (by a small launch ahead of the pass's first attention call) and kept in the plan, checked
 * against the counts before every use: calls that use the same plan must be ordered on the GPU (one
 * stream, or events); use one plan per concurrently decoding batch.
 *
 * Reading ahead of the stream order.  The kernels are launched with programmatic stream
 * serialization.  The first attention call on a stream after fdc_build_masks touches nothing before
 * the kernel ahead of it has completed.  Every later attention call of the pass on that stream
 * reads d_n_active, d_ntiles, d_tiles, d_mask, the plan's work split and the PREFIX rows (rows <
 * prefix_len) of the cache while the kernel ahead of it may still be running; everything else (d_q,
 * the pass's new K/V rows, cache rows >= prefix_len, the workspace, d_out) only after that kernel
 * has completed.  Therefore: (1) the prefix rows of every layer must be complete before the pass's
 * fdc_frontier is reached in stream order, and are never written during decoding; (2) the arrays
 * fdc_frontier / fdc_build_masks produced must not be modified between fdc_build_masks and the last
 * attention call of the pass. */
int fdc_decode_attn(fdc_plan* plan, const fdc_kv_desc* kv, int32_t layer, const int32_t* d_n_active,
                    const uint64_t* d_mask, const int32_t* d_tiles, const int32_t* d_ntiles,
                    const void* d_q, void* d_out, float scale, void* d_workspace, size_t ws_bytes,
                    void* stream);

/* fdc_decode_attn without a workspace argument, for callers that cannot allocate device
 * memory.  (The paper has no counterpart: it describes no memory management at all; this is
 * a deployment variant of the call above and computes exactly the same thing.)
 *
 * Meant for hosts that may not allocate once they run: an in-vehicle runtime whose device
 * memory budget is fixed at start-up and whose decode loop must not call cudaMalloc (it
 * synchronises the device, has no latency bound and fails once the KV pool owns the GPU), or
 * a plugin-style host whose per-step call is forbidden to allocate.  The split partials go
 * to a buffer inside the library image instead: FDC_STATIC_WS_BYTES (16 MiB) of device
 * memory on every GPU that loads the library, held until the process exits.
 *
 *   - Limit: fdc_attn_workspace_bytes(plan, kv) must not exceed FDC_STATIC_WS_BYTES, else
 *     FDC_ERR_STATIC_LIMIT is returned and nothing is launched.  The four bf16/fp32
 *     configurations of up to 16 scenes x 8 KV heads with 64 query rows per KV head fit; 64
 *     scenes x 128 query rows do not.
 *   - The call itself makes no device allocation and frees nothing (no cudaMalloc / cudaFree,
 *     no allocating library routine); inputs and outputs are still the caller's.  Keep
 *     fdc_profile off: profiling creates CUDA events.
 *   - The FIRST call on a device looks up the buffer's device address (a host-side query made
 *     with that device current, checked, then remembered); if nothing of the library has run on
 *     that device yet, the CUDA runtime loads the library's device code at that moment, which
 *     itself takes device memory.  Make that first call during start-up, before any stream
 *     capture is begun; from the second call on the amount of free device memory stays put.  The CUDA device current at the call must
 *     be the plan's device (FDC_ERR_RANGE otherwise).
 *   - All calls on a GPU share the one buffer, and it keeps whatever the last call left.  No
 *     part of it has to start at zero (each call's combine pass reads only partials that the
 *     same call's split pass wrote), so it is never cleared.  Two calls whose kernels can
 *     overlap on the GPU (different streams, or several host threads or plans on one device)
 *     race on it and corrupt each other's results: issue them on one stream or order them
 *     with events. */
int fdc_decode_attn_static(fdc_plan* plan, const fdc_kv_desc* kv, int32_t layer, const int32_t* d_n_active,
                           const uint64_t* d_mask, const int32_t* d_tiles, const int32_t* d_ntiles,
                           const void* d_q, void* d_out, float scale, void* stream);

/* Reads (and with clear != 0 resets, together with the attention kernel's arrival counters,
 * which a launch that gave up may have left behind) the sticky device status word after
 * synchronising `stream`.  *host_bits receives the FDC_DEV_* bits; returns FDC_ERR_DEVICE if non-zero. */
int fdc_status(fdc_plan* plan, int32_t* host_bits, int32_t clear, void* stream);

/* Selects the split-pass kernel: 0 = automatic (3 for bf16, 1 for fp32), 1 = CUDA-core kernel
 * (any dtype), 2 = TMA + mma.sync kernel (bf16), 3 = TMA + tcgen05/TMEM kernel (bf16, head_dim
 * 128; head_dim 64 takes 2).  Unsupported combinations use 1. */
int fdc_set_attn_kernel(fdc_plan* plan, int32_t which);
const char* fdc_kernel_name(int32_t which);

/* Fused append (off by default; Sec. 3.3's shared cache, written and read in one kernel).  While
 * on, an fdc_kv_append on this plan whose cache the tcgen05 attention kernel serves (bf16,
 * head_dim 128) launches nothing: its arguments are recorded, and the NEXT fdc_decode_attn for
 * the same cache, layer, stream and d_n_active writes the rows inside its own kernel, each by
 * the thread block that owns the row's KV tile, before that block loads the tile.  One kernel
 * per layer instead of two dependent ones.  Until that call returns the caller must not read
 * the rows from the cache, and must leave d_n_active, d_kv_row, d_k_new and d_v_new as they
 * were.  Any other call on the plan (another append, an attention call that does not match,
 * fdc_frontier, fdc_build_masks, fdc_state_init, fdc_status, fdc_set_*, fdc_plan_destroy)
 * first launches the recorded append on its own, so no append is ever lost.  Differences from
 * the separate kernel: rows below prefix_len are refused (flagged FDC_DEV_ROW_RANGE like rows
 * >= rows), and a row is written only if its tile is in d_tiles (fdc_build_masks lists it: a
 * new token sees itself). */
int fdc_set_fused_append(fdc_plan* plan, int32_t on);

/* Instrumentation for benchmarks: while enabled, fdc_decode_attn records CUDA events on the
 * launching stream before its split pass, between the passes and after its combine pass (not
 * usable during stream capture).  fdc_profile_read waits for the recorded events, returns
 * the summed durations in milliseconds and the number of recorded calls, and clears the
 * records.  At most 16384 calls are recorded between two reads. */
int fdc_profile(fdc_plan* plan, int32_t enable);
int fdc_profile_read(fdc_plan* plan, float* split_ms, float* combine_ms, int32_t* calls);

/* Algorithm 1's loop test ("while some field is ready") for a decode loop that lives on the
 * device: a CUDA graph whose body is a WHILE conditional node, built by the caller, with one pass
 * of the model as the body (the caller's kernels, fdc_kv_append and fdc_decode_attn per layer,
 * then fdc_frontier and fdc_build_masks for the NEXT pass) and this call as the body's last
 * node.  It launches one thread that
 *   - adds 1 to *d_pass_count (DEVICE int32 [1]; the caller zeroes it before the graph runs:
 *     afterwards it holds the number of passes decoded),
 *   - sets the conditional handle `cond_handle` (a cudaGraphConditionalHandle, created by the
 *     caller for the graph the node belongs to, default value 1) to 1 if *d_all_done == 0
 *     (fdc_frontier's output: some scene still has a ready field) and to 0 otherwise,
 *   - and ends the loop after max_passes passes whatever d_all_done says (FDC_DEV_LOOP_LIMIT is
 *     then set in the status word): a wrong table can never keep the GPU busy for ever.
 * The handle is only meaningful inside a launch of its graph, so the call is for stream capture
 * into the conditional node's body graph (or an explicit kernel node there); launched outside
 * one it fails with a CUDA error at launch or has no effect.  Returns FDC_ERR_NULL / FDC_ERR_RANGE
 * (max_passes < 1) / FDC_ERR_CUDA. */
int fdc_loop_condition(fdc_plan* plan, const int32_t* d_all_done, int32_t* d_pass_count, int32_t max_passes,
                       unsigned long long cond_handle, void* stream);

/* Self-test of the bounded wait that every in-kernel wait of the attention kernels goes through
 * (an mbarrier poll with an iteration limit; when the limit is reached the thread raises its
 * block's abort flag, sets FDC_DEV_TIMEOUT and goes on without waiting).  Launches one block of
 * 64 threads that wait for a barrier nothing will ever complete; the launch ends by itself (about
 * a second), *d_outcome (DEVICE int32 [1]) receives the number of threads whose wait gave up (64)
 * and the plan's status word gets FDC_DEV_TIMEOUT, to be read and cleared with fdc_status.
 * For start-up checks and tests; nothing else in the library calls it. */
int fdc_selftest_bounded_wait(fdc_plan* plan, int32_t* d_outcome, void* stream);

/* Number of kernels this library has launched in the calling process so far. */
int64_t fdc_launch_count(void);

const char* fdc_strerror(int code);
const char* fdc_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FDC_H_ */
