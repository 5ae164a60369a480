// Internal declarations shared by the libcascade translation units (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "cascade.h"

#include <nvtx3/nvToolsExt.h>

// Context: parameters, scratch sized at creation, the sticky device status word.
struct cascade_ctx {
    cascade_params params;
    int device;
    int max_requests;
    int num_sms;
    uint32_t *status_dev;        // sticky CASCADE_ST_* bits
    uint32_t *status_host;       // pinned mirror used by cascade_status
    int cuda_error;              // last failing cudaError_t
    // tier-plan scratch
    unsigned long long *pack_by_slot;  // tier plan: one decision word per request, slot order
    int32_t *want_by_slot;       // plan-first admission: tokens each request is offered (budget -> schedule)
    int4 *work_admit;            // per admitted request: slot, pop offset, restore offset, counts
    int4 *work_victim;           // per preempted request: slot, freed offset, evict offset, action
    int32_t *plan_scalars;       // device scalars handed from the plan kernel to the apply kernels
    int max_cluster;             // largest cluster the device co-schedules for the cluster kernels
    int sort_cluster;            // cluster size override for the ordering kernel (0 = automatic)
    int sort_items;              // keys per thread override (0 = automatic)
    int sort_threads;            // threads per CTA override (0 = automatic)
    int sort_stage;              // 1: group elements by digit locally before the remote scatter
    int sort_async;              // 1: per-pass exchanges complete on mbarriers instead of cluster barriers
    int copy_ctas_host;          // copy CTAs per SM when the record pool is pinned host memory
    int copy_ctas_dev;           // copy CTAs per SM when the record pool is device memory
    int copy_bulk_host;          // >0: TMA bulk-copy ring (that many CTAs per SM) for the pinned-host path
    int copy_bulk_dev;           // >0: TMA bulk-copy ring for the device-staging path
    int move_ctas;               // >0: CTAs of each of the two grids of the fused evict+restore (at most half the SMs)
    int copy_grid_host;          // >0: CTAs of the TMA ring over the host link (default: 44 % of the SMs)
    int move_ctas_restore;       // >0: SMs' worth of CTAs of the restore grid alone (tuning)
    int move_vector;             // fused move: bit 0 = restore grid, bit 1 = evict grid use the vector kernel instead of the ring
    int copy_ahead_sub;          // TMA ring: loads kept in flight = ring slots minus this (1 | 2)
    int copy_piece;              // >0: piece size in bytes of the TMA ring (8192 | 16384 | 32768); 0 = picked per call
    int copy_ring_kb;            // >0: shared memory of the TMA ring in KiB (64..128); 0 = 128 (host) / 96 (device)
    int copy_dynamic;            // 1: the TMA ring hands its pieces out on demand (a counter) instead of by a fixed stride
    unsigned *copy_tickets;      // device: 64 pairs of counters, one pair per launch of the ring kernel in turn, zero between uses
    unsigned copy_ticket_seq;    // launches so far
    int pdl;                     // 1: programmatic dependent launch between the calls' kernels
    void *sort_runs, *sort_sorted;   // queues beyond 32768 requests: the ordered runs and the merged order (16 B per request each)
    int multi_sort;              // 1: such queues are ordered as runs of 16384 by one cluster each, then merged by rank
    int plan_prepare_min;        // queues above this size run the tier plan's per-request phase as a grid of its own
    int sort_top_first;          // 1: radix passes over key bits 32..63 only, then equal values are put in order of the low bits (budget policy only)
    int merge_sort;              // 1: queues beyond the counting path that fit one key per thread (up to 4096) are ordered by local sort + merge by rank; 2: every queue of up to 16384
    int rank_sort_max;           // queues up to this size are ordered by counting instead of radix passes
    // copy-engine path (cascade_kv_move_staged): side streams and events, created with the context
    cudaStream_t ce_stream[4];   // [0], [1] host -> staging (restores); [2], [3] staging -> host (evictions)
    cudaEvent_t ce_event[7];     // lists published, gather done, scatter done, fill done x2, drain done x2
    int ce_lanes;                // side streams used per direction (1 | 2)
    unsigned long long *ce_bitmap;   // host-side: one bit per host record, grown on demand
    size_t ce_bitmap_words;
    int test_move_stall;         // test hooks (CASCADE_TEST_MOVE_STALL): 1 = the evict side of the fused move never
                                 // reports a block as read out, 2 = the first piece of CTA 0 of a ring kernel announces
                                 // more bytes than it loads; both make a bounded wait run out; 1, 2 and 3 lower the
                                 // limit of every bounded wait of the copy kernels to a tenth of a second
};

// plan_scalars layout
enum { PS_N_ADMIT = 0, PS_N_VICTIM, PS_HBM_CNT0, PS_HOST_CNT0, PS_TOTAL_FREED, PS_COUNT };

// NVTX range around the launches of one entry point (visible in Nsight timelines; a no-op without a tool)
struct CascadeRange {
    explicit CascadeRange(const char *name) { nvtxRangePushA(name); }
    ~CascadeRange() { nvtxRangePop(); }
};

#define CASCADE_CUDA_TRY(ctx, expr)                         \
    do {                                                    \
        cudaError_t e__ = (expr);                           \
        if (e__ != cudaSuccess) {                           \
            (ctx)->cuda_error = (int)e__;                   \
            return CASCADE_ECUDA;                           \
        }                                                   \
    } while (0)

// ---- the integer cost model, device side --------------------------------------------------
// Load-dependent constants are folded on the host once per call (exact integer arithmetic).
struct LoadConsts {
    int64_t A_act, A_max;          // per-token prefill cost under actual / maximum load (Q20 ns)
    int64_t dec_act, dec_max;      // iteration cost with one more decode sequence, before its KV term,
                                   // plus a full prefill chunk (Q20 ns)
};

static inline int64_t host_iter_q(const cascade_params &p, int64_t D, int64_t K) {
    return p.c_iter_q20 + D * p.c_dseq_q20 + K * p.c_dkv_q20;
}

static inline LoadConsts make_load_consts(const cascade_params &p, int32_t D_act, int64_t K_act) {
    int64_t Dm = D_act > p.max_batch - 1 ? D_act : p.max_batch - 1;
    int64_t Kcap = (int64_t)(p.max_batch - 1) * p.max_ctx_avg;
    int64_t Km = K_act > Kcap ? K_act : Kcap;
    LoadConsts c;
    c.A_act = p.c_tok_q20 + (host_iter_q(p, D_act, K_act) >> p.chunk_shift);
    c.A_max = p.c_tok_q20 + (host_iter_q(p, Dm, Km) >> p.chunk_shift);
    int64_t chunk_q = p.c_tok_q20 << p.chunk_shift;
    c.dec_act = host_iter_q(p, (int64_t)D_act + 1, K_act) + chunk_q;
    c.dec_max = host_iter_q(p, Dm + 1, Km) + chunk_q;
    return c;
}

__device__ __forceinline__ int64_t dev_comp_q(int64_t A, int64_t c_attn, int64_t P, int64_t s) {
    return A * (P - s) + c_attn * (P * P - s * s);
}

__device__ __forceinline__ int64_t dev_restore_time(const cascade_params &p, int k, int64_t x) {
    return x == 0 ? 0 : p.delta_ns[k] + x * p.blk_ns[k];
}

__device__ __forceinline__ bool dev_request_valid(int32_t bt, int64_t P, int64_t n0, int64_t n1, int64_t n2) {
    if (P < 1 || P > (int64_t(1) << 17)) return false;
    if ((n0 | n1 | n2) < 0) return false;
    int64_t h = n0 + n1 + n2;
    if (h > (int64_t(1) << 13)) return false;
    return h * bt < P;
}

// Geometry of the two cluster kernels (ordering and tier plan): T threads per CTA, K elements per
// thread, C CTAs per cluster, C*T*K >= n and T*K <= 4096.  Chosen by measurement on B200; the
// context's overrides (environment, for tuning) win when they are consistent.
static inline bool cascade_pick_geometry(const cascade_ctx *ctx, int n, int *T, int *C, int *K) {
    int t, c, k;
    if (n <= 1024) { t = 256; c = 4; k = 1; }
    else if (n <= 2048) { t = 256; c = 8; k = 1; }
    else if (n <= 4096) { t = 256; c = 16; k = 1; }
    else if (n <= 8192) { t = 256; c = 16; k = 2; }
    else if (n <= 16384) { t = 256; c = 16; k = 4; }
    else if (n <= 32768) { t = 512; c = 16; k = 4; }
    else { t = 512; c = 16; k = 8; }
    if (ctx->sort_threads == 256 || ctx->sort_threads == 512) t = ctx->sort_threads;
    if (ctx->sort_items == 1 || ctx->sort_items == 2 || ctx->sort_items == 4 || ctx->sort_items == 8)
        k = ctx->sort_items;
    if (ctx->sort_cluster == 1 || ctx->sort_cluster == 2 || ctx->sort_cluster == 4 || ctx->sort_cluster == 8 ||
        ctx->sort_cluster == 16)
        c = ctx->sort_cluster;
    // a device that cannot co-schedule the preferred cluster gets a smaller one with more keys per CTA
    const int cmax = ctx->max_cluster > 0 ? ctx->max_cluster : 16;
    while (c > cmax && c > 1) {
        c /= 2;
        if (k < 8) k *= 2; else if (t < 512) t = 512;
    }
    *T = t; *C = c; *K = k;
    return (long long)c * t * k >= n && t * k <= 4096;
}

// The Eq. 7 bounds (host first, deep tier from what is left and only behind a fully restored host
// segment) and the endpoint candidate with the smallest predicted completion time; ties restore more.
__device__ __forceinline__ void dev_choose_restore(const cascade_params &p, int64_t A_act, int64_t P, int64_t n0,
                                                   int64_t n1, int64_t n2, int64_t budget, int64_t *x1, int64_t *x2) {
    const int64_t rem = budget > 0 ? budget : 0;
    const int64_t bt = p.bt;
    int64_t x1max = 0;
    if (n1 > 0) {
        int64_t head = rem - p.delta_ns[1];
        if (head < 0) head = 0;
        x1max = head / p.blk_ns[1];
        if (x1max > n1) x1max = n1;
    }
    int64_t x2max = 0;
    if (x1max == n1 && n2 > 0) {
        int64_t head = rem - dev_restore_time(p, 1, n1) - p.delta_ns[2];
        if (head < 0) head = 0;
        x2max = head / p.blk_ns[2];
        if (x2max > n2) x2max = n2;
    }
    int64_t bx1 = 0, bx2 = 0;
    int64_t bF = dev_comp_q(A_act, p.c_attn_q20, P, n0 * bt);
    if (x1max > 0) {
        const int64_t F = (dev_restore_time(p, 1, x1max) << 20) + dev_comp_q(A_act, p.c_attn_q20, P, (n0 + x1max) * bt);
        if (F <= bF) { bF = F; bx1 = x1max; }
    }
    if (x2max > 0) {
        const int64_t F = ((dev_restore_time(p, 1, n1) + dev_restore_time(p, 2, x2max)) << 20) +
                          dev_comp_q(A_act, p.c_attn_q20, P, (n0 + n1 + x2max) * bt);
        if (F <= bF) { bF = F; bx1 = n1; bx2 = x2max; }
    }
    *x1 = bx1;
    *x2 = bx2;
}

// ---- programmatic dependent launch -----------------------------------------------------------
// Every kernel of the path starts with cascade_grid_wait(): launched with the programmatic
// stream-serialization attribute it may be scheduled while its predecessor in the stream is still
// running and blocks here until that grid has completed and its writes are visible; launched
// without the attribute the instruction does nothing.  The short plan kernels then call
// cascade_grid_trigger() at once, so that the launch latency of the next kernel overlaps their own
// run time; the long copy kernels never trigger early (their successor starts when they exit).
// No kernel touches global memory before the wait, and every thread executes it (also threads that
// return right after), so completion of a grid implies completion of everything before it.
__device__ __forceinline__ void cascade_grid_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void cascade_grid_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t cascade_launch(bool pdl, int cluster, dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                         void (*kernel)(KArgs...), Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned na = 0;
    if (cluster > 0) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = cluster;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args &&>(args)...);
}

// Function attributes (shared-memory opt-in, non-portable cluster size) are set once per device and kernel.  The flag may
// be read and written by several host threads: setting an attribute twice is harmless, so a set-once atomic is enough.
struct CascadeDeviceOnce {
    std::atomic<bool> done[64] = {};
    bool is_set(int device) const { return device >= 0 && device < 64 && done[device].load(std::memory_order_acquire); }
    void set(int device) {
        if (device >= 0 && device < 64) done[device].store(true, std::memory_order_release);
    }
};

// The hot calls launch on the calling thread's current device and dereference the context's allocations there:
// a context of another device is rejected on the host (CASCADE_EINVAL) before anything is launched.
static inline bool cascade_on_ctx_device(const cascade_ctx *ctx) {
    int d = -1;
    return cudaGetDevice(&d) == cudaSuccess && d == ctx->device;
}

// entry points implemented in the other translation units
int cascade_validate_params(const cascade_params *p);
int cascade_probe_max_cluster();
