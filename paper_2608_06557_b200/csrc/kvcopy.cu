// cascade_kv_restore / cascade_kv_evict: paged KV-block copies between a record-major pool
// (pinned host memory read or written over the host link, or a device staging buffer) and the
// paged HBM pool, driven by (src id, dst id) lists that live in device memory.
//
// The bytes are opaque.  A block is n_chunks pieces of chunk_bytes; on the record side they are
// back to back, on the HBM side chunk c of block b sits at c*chunk_stride + b*block_stride.
// Two kernels do the same copy:
//   kv_copy_bulk_kernel (default)  one elected thread per CTA drives TMA bulk copies
//       (cp.async.bulk) through a 4-slot shared-memory ring, 32 KiB pieces, one or two CTAs per SM;
//       it leaves the SMs' issue slots free for whatever else runs on the GPU;
//   kv_copy_kernel                 256 threads x 4 x 16-byte vector loads/stores per 16 KiB piece on a
//       persistent grid (selected with CASCADE_COPY_BULK_HOST=0 / CASCADE_COPY_BULK_DEV=0).
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;
constexpr int kPiece = kThreads * kUnroll * 16;  // bytes moved by one CTA iteration

struct CopyArgs {
    char *paged;              // HBM pool base
    char *record;             // record-major pool base
    const int32_t *src_ids;
    const int32_t *dst_ids;
    const int32_t *n_dev;     // device count or NULL
    uint32_t *status;
    long long paged_blocks, record_blocks;
    long long chunk_bytes, chunk_stride, block_stride;
    int n_chunks;
    int n_max;
    int pieces_per_chunk;
};

template <bool kRestore>
__global__ void __launch_bounds__(kThreads) kv_copy_kernel(const __grid_constant__ CopyArgs a) {
    cascade_grid_wait();
    int count = a.n_max;
    if (a.n_dev) {
        const int c = *a.n_dev;
        count = c < 0 ? 0 : (c < count ? c : count);
    }
    const long long per_block = (long long)a.n_chunks * a.pieces_per_chunk;
    const long long items = (long long)count * per_block;
    const long long bb = (long long)a.n_chunks * a.chunk_bytes;
    const int tid = threadIdx.x;
    bool bad = false;
    for (long long it = blockIdx.x; it < items; it += gridDim.x) {
        const long long i = it / per_block;
        const int rem = (int)(it - i * per_block);
        const int c = rem / a.pieces_per_chunk;
        const int pc = rem - c * a.pieces_per_chunk;
        const long long s = a.src_ids[i], d = a.dst_ids[i];
        const long long rec_id = kRestore ? s : d, pg_id = kRestore ? d : s;
        if (rec_id < 0 || rec_id >= a.record_blocks || pg_id < 0 || pg_id >= a.paged_blocks) {
            bad = true;  // id outside its pool: this pair is skipped
            continue;
        }
        char *rec = a.record + rec_id * bb + (long long)c * a.chunk_bytes;
        char *pg = a.paged + (long long)c * a.chunk_stride + pg_id * a.block_stride;
        const char *src = kRestore ? rec : pg;
        char *dst = kRestore ? pg : rec;
        const long long base = (long long)pc * kPiece + tid * 16;
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const long long off = base + (long long)u * kThreads * 16;
            if (off < a.chunk_bytes) v[u] = __ldcs(reinterpret_cast<const uint4 *>(src + off));
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const long long off = base + (long long)u * kThreads * 16;
            if (off < a.chunk_bytes) __stcs(reinterpret_cast<uint4 *>(dst + off), v[u]);
        }
    }
    if (bad && tid == 0) atomicOr(a.status, CASCADE_ST_EBOUNDS);
}


// ---- bulk-copy variant: TMA (cp.async.bulk) through a shared-memory ring ---------------------------
// One elected thread per CTA moves pieces of up to 32 KiB: global -> shared with an mbarrier that
// counts the arriving bytes, then shared -> global as a bulk store group.  kStages ring slots; two
// loads are kept in flight ahead of the piece being stored, and a slot is refilled only after the
// store that last used it has finished reading shared memory.  Every wait is bounded: when the
// clock limit is hit the kernel records CASCADE_ST_ETIMEOUT, stops issuing work, drains its own
// store groups and returns.
constexpr int kBulkPiece = 32 * 1024;
constexpr int kStages = 4;
constexpr int kAhead = kStages - 2;
constexpr long long kWaitCycles = 4000000000LL;  // about two seconds at 1.9 GHz

__device__ __forceinline__ unsigned smem_addr(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_load(unsigned dst_smem, const void *src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, unsigned src_smem, unsigned bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

template <bool kRestore>
__global__ void __launch_bounds__(32) kv_copy_bulk_kernel(const __grid_constant__ CopyArgs a) {
    cascade_grid_wait();
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) unsigned long long bars[kStages];
    if (threadIdx.x != 0) return;
    for (int s = 0; s < kStages; ++s) mbar_init(smem_addr(&bars[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    int count = a.n_max;
    if (a.n_dev) {
        const int c = *a.n_dev;
        count = c < 0 ? 0 : (c < count ? c : count);
    }
    const int ppc = a.pieces_per_chunk;  // pieces of kBulkPiece per chunk
    const long long per_block = (long long)a.n_chunks * ppc;
    const long long items = (long long)count * per_block;
    const long long bb = (long long)a.n_chunks * a.chunk_bytes;
    uint32_t st = 0;

    long long next = blockIdx.x;  // next item of this CTA to load
    // resolves item `it` into addresses; false when an id is outside its pool (pair skipped)
    auto resolve = [&](long long it, const char *&src, char *&dst, unsigned &bytes) -> bool {
        const long long i = it / per_block;
        const int rem = (int)(it - i * per_block);
        const int c = rem / ppc, pc = rem - c * ppc;
        const long long s = a.src_ids[i], d = a.dst_ids[i];
        const long long rec_id = kRestore ? s : d, pg_id = kRestore ? d : s;
        if (rec_id < 0 || rec_id >= a.record_blocks || pg_id < 0 || pg_id >= a.paged_blocks) return false;
        const long long off = (long long)pc * kBulkPiece;
        const long long left = a.chunk_bytes - off;
        bytes = (unsigned)(left < kBulkPiece ? left : kBulkPiece);
        char *rec = a.record + rec_id * bb + (long long)c * a.chunk_bytes + off;
        char *pg = a.paged + (long long)c * a.chunk_stride + pg_id * a.block_stride + off;
        src = kRestore ? rec : pg;
        dst = kRestore ? pg : rec;
        return true;
    };
    char *dst_of[kStages];
    unsigned bytes_of[kStages];
    long long issued = 0, stored = 0;
    auto issue_next = [&]() -> bool {  // loads the next valid item into ring slot issued % kStages
        while (next < items) {
            const char *src;
            char *dst;
            unsigned bytes;
            const bool ok = resolve(next, src, dst, bytes);
            next += gridDim.x;
            if (!ok) {
                st |= CASCADE_ST_EBOUNDS;
                continue;
            }
            const int slot = (int)(issued % kStages);
            const unsigned bar = smem_addr(&bars[slot]);
            mbar_expect_tx(bar, bytes);
            bulk_load(smem_addr(ring + (size_t)slot * kBulkPiece), src, bytes, bar);
            dst_of[slot] = dst;
            bytes_of[slot] = bytes;
            ++issued;
            return true;
        }
        return false;
    };
    for (int k = 0; k < kAhead; ++k)
        if (!issue_next()) break;
    while (stored < issued) {
        const int slot = (int)(stored % kStages);
        const unsigned parity = (unsigned)((stored / kStages) & 1);
        const unsigned bar = smem_addr(&bars[slot]);
        const long long t0 = clock64();
        bool arrived = mbar_try_wait(bar, parity);
        while (!arrived && clock64() - t0 < kWaitCycles) arrived = mbar_try_wait(bar, parity);
        if (!arrived) {  // give up: record it, issue nothing more
            st |= CASCADE_ST_ETIMEOUT;
            break;
        }
        bulk_store(dst_of[slot], smem_addr(ring + (size_t)slot * kBulkPiece), bytes_of[slot]);
        ++stored;
        // the slot refilled next was last read by the store issued one step earlier
        asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        issue_next();
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (st) atomicOr(a.status, st);
}

// ---- fused evict + restore ("move"): both directions of the host link at once ----------------------
// The evict list and the restore list of one iteration in ONE ring kernel.  Evicted blocks travel
// device -> host while restored blocks travel host -> device, so the link is used in both directions
// at the same time.  A restore may target an HBM block that the same call evicts (the tier plan hands
// freed blocks out again at once): its store into HBM waits until every piece of that block has been
// read by the evict side.  Each CTA works on one list: the CTAs are shared out in proportion to the
// lists' lengths; evict CTAs walk their list backwards, because the blocks freed last are handed out
// first.  Only restore CTAs ever wait, and
// only for evict CTAs, which never wait for anybody, so with all CTAs resident (one per SM at most)
// the waits cannot deadlock.  They are clock-bounded all the same (CASCADE_ST_ETIMEOUT, that store
// is skipped).
struct MoveArgs {
    char *paged;
    char *record;
    const int32_t *evict_src, *evict_dst, *restore_src, *restore_dst;
    const int32_t *n_evict_dev, *n_restore_dev;
    int32_t *dep;    // per restore: index into the evict list of the entry that frees its HBM block, or -1
    int32_t *done;   // per evict entry: pieces of the block already read out of HBM
    uint32_t *status;
    long long paged_blocks, record_blocks;
    long long chunk_bytes, chunk_stride, block_stride;
    int n_chunks;
    int n_evict_max, n_restore_max;
    int pieces_per_chunk;
    int stall;       // test hook: the evict side never reports a block as read out (exercises the bounded wait)
};

__device__ __forceinline__ int clamp_count(const int32_t *dev, int maxv) {
    if (!dev) return maxv;
    const int c = *dev;
    return c < 0 ? 0 : (c < maxv ? c : maxv);
}

__global__ void __launch_bounds__(256) kv_move_prepare_kernel(const __grid_constant__ MoveArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int ne = clamp_count(a.n_evict_dev, a.n_evict_max), nr = clamp_count(a.n_restore_dev, a.n_restore_max);
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int stride = gridDim.x * blockDim.x;
    for (int j = i; j < ne; j += stride) a.done[j] = 0;
    for (int r = i; r < nr; r += stride) {
        const int32_t g = a.restore_dst[r];
        int dep = -1;
        for (int j = 0; j < ne; ++j)
            if (a.evict_src[j] == g) dep = j;
        a.dep[r] = dep;
    }
}

__global__ void __launch_bounds__(32) kv_move_kernel(const __grid_constant__ MoveArgs a) {
    cascade_grid_wait();
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) unsigned long long bars[kStages];
    if (threadIdx.x != 0) return;
    for (int s = 0; s < kStages; ++s) mbar_init(smem_addr(&bars[s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    const int ne = clamp_count(a.n_evict_dev, a.n_evict_max), nr = clamp_count(a.n_restore_dev, a.n_restore_max);
    const int ppc = a.pieces_per_chunk;
    const long long per_block = (long long)a.n_chunks * ppc;
    const long long bb = (long long)a.n_chunks * a.chunk_bytes;
    uint32_t st = 0;
    // Each CTA serves one direction, so that both directions of the link are busy at once; the CTAs are shared
    // out in proportion to the bytes of the two lists (interleaved over the grid), at least one per non-empty
    // list.  A single-CTA grid does the evict list first, then the restores.
    const long long G = gridDim.x, b = blockIdx.x;
    const bool both = G == 1;                          // one CTA walks both lists
    long long ge = G;                                  // CTAs that evict
    if (ne > 0 && nr > 0) {
        ge = (G * ne + (ne + (long long)nr) / 2) / (ne + (long long)nr);
        ge = ge < 1 ? 1 : (ge > G - 1 ? G - 1 : ge);
    } else if (ne == 0) {
        ge = 0;
    }
    const long long e_before = b * ge / G;             // evict CTAs among the blocks before this one
    const bool evict_role = (b + 1) * ge / G > e_before;
    const long long evict_items = (both || evict_role) ? (long long)ne * per_block : 0;
    const long long items = evict_items + ((both || !evict_role) ? (long long)nr * per_block : 0);
    const long long step = both ? 1 : (evict_role ? ge : G - ge);

    long long next = both ? 0 : (evict_role ? e_before : b - e_before);
    char *dst_of[kStages];
    unsigned bytes_of[kStages];
    int evict_of[kStages];  // evict-list index to signal after the load (evict piece), -1 otherwise
    int wait_of[kStages];   // evict-list index to wait for before the store (restore piece), -1 if none
    long long issued = 0, stored = 0;
    auto issue_next = [&]() -> bool {
        while (next < items) {
            const long long it = next;
            next += step;
            const bool is_evict = it < evict_items;
            const long long local = is_evict ? it : it - evict_items;
            long long i = local / per_block;
            const int rem = (int)(local - i * per_block);
            if (is_evict) i = ne - 1 - i;  // blocks freed last are reused first: read them out first
            const int c = rem / ppc, pc = rem - c * ppc;
            const long long rec_id = is_evict ? a.evict_dst[i] : a.restore_src[i];
            const long long pg_id = is_evict ? a.evict_src[i] : a.restore_dst[i];
            if (rec_id < 0 || rec_id >= a.record_blocks || pg_id < 0 || pg_id >= a.paged_blocks) {
                st |= CASCADE_ST_EBOUNDS;
                // a skipped evict piece still counts as read, or a restore into that block would wait for nothing
                if (is_evict) atomicAdd(&a.done[i], 1);
                continue;
            }
            const long long off = (long long)pc * kBulkPiece;
            const long long left = a.chunk_bytes - off;
            const unsigned bytes = (unsigned)(left < kBulkPiece ? left : kBulkPiece);
            char *rec = a.record + rec_id * bb + (long long)c * a.chunk_bytes + off;
            char *pg = a.paged + (long long)c * a.chunk_stride + pg_id * a.block_stride + off;
            const int slot = (int)(issued % kStages);
            const unsigned bar = smem_addr(&bars[slot]);
            mbar_expect_tx(bar, bytes);
            bulk_load(smem_addr(ring + (size_t)slot * kBulkPiece), is_evict ? pg : rec, bytes, bar);
            dst_of[slot] = is_evict ? rec : pg;
            bytes_of[slot] = bytes;
            evict_of[slot] = is_evict ? (int)i : -1;
            wait_of[slot] = is_evict ? -1 : a.dep[i];
            ++issued;
            return true;
        }
        return false;
    };
    for (int k = 0; k < kAhead; ++k)
        if (!issue_next()) break;
    while (stored < issued) {
        const int slot = (int)(stored % kStages);
        const unsigned parity = (unsigned)((stored / kStages) & 1);
        const unsigned bar = smem_addr(&bars[slot]);
        long long t0 = clock64();
        bool arrived = mbar_try_wait(bar, parity);
        while (!arrived && clock64() - t0 < kWaitCycles) arrived = mbar_try_wait(bar, parity);
        if (!arrived) {
            st |= CASCADE_ST_ETIMEOUT;
            break;
        }
        bool skip = false;
        if (evict_of[slot] >= 0) {
            if (!a.stall) atomicAdd(&a.done[evict_of[slot]], 1);  // this piece of the block has left HBM
        } else if (wait_of[slot] >= 0) {
            // the HBM block is being evicted by this same call: write only after it has been read out
            const volatile int32_t *flag = a.done + wait_of[slot];
            t0 = clock64();
            if (st & CASCADE_ST_ETIMEOUT) skip = true;  // one expired wait is enough: do not queue up more
            const long long limit = a.stall ? kWaitCycles / 20 : kWaitCycles;
            while (!skip && *flag < (int)per_block) {
                if (clock64() - t0 > limit) {
                    st |= CASCADE_ST_ETIMEOUT;
                    skip = true;
                    break;
                }
            }
            __threadfence();
        }
        if (!skip) bulk_store(dst_of[slot], smem_addr(ring + (size_t)slot * kBulkPiece), bytes_of[slot]);
        ++stored;
        asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        issue_next();
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (st) atomicOr(a.status, st);
}

int check_layout(const cascade_kv_layout *l, const void *paged, const void *record, long long record_blocks) {
    if (!l || !paged || !record) return CASCADE_EINVAL;
    if (l->n_blocks < 0 || record_blocks < 0 || l->n_chunks < 1 || l->chunk_bytes < 16) return CASCADE_EINVAL;
    if ((l->chunk_bytes | l->chunk_stride | l->block_stride) & 15) return CASCADE_EINVAL;
    if (l->chunk_stride < 0 || l->block_stride < 0) return CASCADE_EINVAL;
    if (((uintptr_t)paged | (uintptr_t)record) & 15) return CASCADE_EINVAL;
    return CASCADE_OK;
}

template <bool kRestore>
int launch_copy(cascade_ctx *ctx, const cascade_kv_layout *l, char *paged, char *record, long long record_blocks,
                int record_is_device, const int32_t *src_ids, const int32_t *dst_ids, const int32_t *n_dev, int n_max,
                cudaStream_t s) {
    if (!ctx || n_max < 0) return CASCADE_EINVAL;
    if (n_max == 0) return CASCADE_OK;
    int rc = check_layout(l, paged, record, record_blocks);
    if (rc != CASCADE_OK) return rc;
    if (!src_ids || !dst_ids) return CASCADE_EINVAL;
    CopyArgs a;
    a.paged = paged;
    a.record = record;
    a.src_ids = src_ids;
    a.dst_ids = dst_ids;
    a.n_dev = n_dev;
    a.status = ctx->status_dev;
    a.paged_blocks = l->n_blocks;
    a.record_blocks = record_blocks;
    a.chunk_bytes = l->chunk_bytes;
    a.chunk_stride = l->chunk_stride;
    a.block_stride = l->block_stride;
    a.n_chunks = l->n_chunks;
    a.n_max = n_max;
    const int mode = record_is_device ? ctx->copy_bulk_dev : ctx->copy_bulk_host;
    if (mode) {
        // TMA ring: one CTA (one elected thread) per SM slot, 32 KiB pieces
        a.pieces_per_chunk = (int)((l->chunk_bytes + kBulkPiece - 1) / kBulkPiece);
        const long long items = (long long)n_max * l->n_chunks * a.pieces_per_chunk;
        long long grid = (long long)ctx->num_sms * (mode > 1 ? mode : 1);
        if (grid > items) grid = items;
        const size_t smem = (size_t)kStages * kBulkPiece;
        static bool configured_dev[64] = {};
        bool unknown = false;
        bool &configured = (ctx->device >= 0 && ctx->device < 64) ? configured_dev[ctx->device] : unknown;
        if (!configured) {
            CASCADE_CUDA_TRY(ctx, cudaFuncSetAttribute(kv_copy_bulk_kernel<true>,
                                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            CASCADE_CUDA_TRY(ctx, cudaFuncSetAttribute(kv_copy_bulk_kernel<false>,
                                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            configured = true;
        }
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)grid), dim3(32), smem, s,
                                             kv_copy_bulk_kernel<kRestore>, a));
        return CASCADE_OK;
    }
    a.pieces_per_chunk = (int)((l->chunk_bytes + kPiece - 1) / kPiece);
    const long long items = (long long)n_max * l->n_chunks * a.pieces_per_chunk;
    const int per_sm = record_is_device ? ctx->copy_ctas_dev : ctx->copy_ctas_host;
    long long grid = (long long)ctx->num_sms * per_sm;
    if (grid > items) grid = items;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)grid), dim3(kThreads), 0, s, kv_copy_kernel<kRestore>, a));
    return CASCADE_OK;
}

}  // namespace

extern "C" int cascade_kv_restore(cascade_ctx *ctx, const cascade_kv_layout *hbm, void *hbm_pool, const void *src_pool,
                                  int64_t src_blocks, int src_is_device, const int32_t *src_ids,
                                  const int32_t *dst_ids, const int32_t *n_copies_dev, int n_copies_max,
                                  void *stream) {
    CascadeRange nvtx_range("cascade_kv_restore");
    return launch_copy<true>(ctx, hbm, (char *)hbm_pool, (char *)const_cast<void *>(src_pool), src_blocks,
                             src_is_device, src_ids, dst_ids, n_copies_dev, n_copies_max, (cudaStream_t)stream);
}

extern "C" int cascade_kv_evict(cascade_ctx *ctx, const cascade_kv_layout *hbm, const void *hbm_pool, void *dst_pool,
                                int64_t dst_blocks, int dst_is_device, const int32_t *src_ids, const int32_t *dst_ids,
                                const int32_t *n_copies_dev, int n_copies_max, void *stream) {
    CascadeRange nvtx_range("cascade_kv_evict");
    return launch_copy<false>(ctx, hbm, (char *)const_cast<void *>(hbm_pool), (char *)dst_pool, dst_blocks,
                              dst_is_device, src_ids, dst_ids, n_copies_dev, n_copies_max, (cudaStream_t)stream);
}

// Deep-tier record -> host record: the bulk-copy ring with a "paged" side that is itself record-major
// (one chunk per record).
extern "C" int cascade_kv_stage(cascade_ctx *ctx, const void *deep_pool, int64_t deep_blocks, void *host_pool,
                                int64_t host_blocks, int64_t block_bytes, const int32_t *src_ids,
                                const int32_t *dst_ids, const int32_t *n_copies_dev, int n_copies_max, void *stream) {
    CascadeRange nvtx_range("cascade_kv_stage");
    if (block_bytes < 16 || (block_bytes & 15) || host_blocks < 0) return CASCADE_EINVAL;
    cascade_kv_layout rec;
    rec.n_blocks = host_blocks;
    rec.n_chunks = 1;
    rec.reserved = 0;
    rec.chunk_bytes = block_bytes;
    rec.chunk_stride = block_bytes;
    rec.block_stride = block_bytes;
    return launch_copy<true>(ctx, &rec, (char *)host_pool, (char *)const_cast<void *>(deep_pool), deep_blocks, 0,
                             src_ids, dst_ids, n_copies_dev, n_copies_max, (cudaStream_t)stream);
}

extern "C" int cascade_kv_move(cascade_ctx *ctx, const cascade_kv_layout *hbm, void *hbm_pool, void *host_pool,
                               int64_t host_blocks, const int32_t *evict_src, const int32_t *evict_dst,
                               const int32_t *n_evict_dev, int n_evict_max, const int32_t *restore_src,
                               const int32_t *restore_dst, const int32_t *n_restore_dev, int n_restore_max,
                               int32_t *scratch, void *stream) {
    CascadeRange nvtx_range("cascade_kv_move");
    if (!ctx || n_evict_max < 0 || n_restore_max < 0) return CASCADE_EINVAL;
    if (n_evict_max == 0 && n_restore_max == 0) return CASCADE_OK;
    int rc = check_layout(hbm, hbm_pool, host_pool, host_blocks);
    if (rc != CASCADE_OK) return rc;
    if (!scratch || (n_evict_max > 0 && (!evict_src || !evict_dst)) || (n_restore_max > 0 && (!restore_src || !restore_dst)))
        return CASCADE_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    MoveArgs a;
    a.paged = (char *)hbm_pool;
    a.record = (char *)host_pool;
    a.evict_src = evict_src;
    a.evict_dst = evict_dst;
    a.restore_src = restore_src;
    a.restore_dst = restore_dst;
    a.n_evict_dev = n_evict_dev;
    a.n_restore_dev = n_restore_dev;
    a.dep = scratch;
    a.done = scratch + n_restore_max;
    a.status = ctx->status_dev;
    a.paged_blocks = hbm->n_blocks;
    a.record_blocks = host_blocks;
    a.chunk_bytes = hbm->chunk_bytes;
    a.chunk_stride = hbm->chunk_stride;
    a.block_stride = hbm->block_stride;
    a.n_chunks = hbm->n_chunks;
    a.n_evict_max = n_evict_max;
    a.n_restore_max = n_restore_max;
    a.pieces_per_chunk = (int)((hbm->chunk_bytes + kBulkPiece - 1) / kBulkPiece);
    a.stall = ctx->test_move_stall;
    const int most = n_evict_max > n_restore_max ? n_evict_max : n_restore_max;
    int pgrid = (most + 255) / 256;
    if (pgrid > ctx->num_sms * 4) pgrid = ctx->num_sms * 4;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(pgrid), dim3(256), 0, s, kv_move_prepare_kernel, a));
    const long long items = ((long long)n_evict_max + n_restore_max) * hbm->n_chunks * a.pieces_per_chunk;
    long long grid = ctx->num_sms;  // one resident CTA per SM: every CTA that can be waited for is running
    if (ctx->move_ctas > 0 && ctx->move_ctas < grid) grid = ctx->move_ctas;
    if (grid > items) grid = items;
    const size_t smem = (size_t)kStages * kBulkPiece;
    static bool configured_dev[64] = {};
    bool unknown = false;
    bool &configured = (ctx->device >= 0 && ctx->device < 64) ? configured_dev[ctx->device] : unknown;
    if (!configured) {
        CASCADE_CUDA_TRY(ctx, cudaFuncSetAttribute(kv_move_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured = true;
    }
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)grid), dim3(32), smem, s, kv_move_kernel, a));
    return CASCADE_OK;
}
