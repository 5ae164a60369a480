// cascade_kv_restore / cascade_kv_evict / cascade_kv_move / cascade_kv_stage: paged KV-block copies
// between a record-major pool (pinned host memory read or written over the host link, or a device
// staging buffer) and the paged HBM pool, driven by (src id, dst id) lists that live in device memory.
//
// The bytes are opaque.  A block is n_chunks pieces of chunk_bytes; on the record side they are
// back to back, on the HBM side chunk c of block b sits at c*chunk_stride + b*block_stride.
// Two kernels do the same copy:
//   kv_ring_kernel (default)  one elected thread per CTA drives TMA bulk copies (cp.async.bulk)
//       through a shared-memory ring; the piece size (8, 16 or 32 KiB) is picked per call from the
//       number of blocks actually moved, so that a call of one block still spreads over the grid;
//       it leaves the SMs' issue slots free for whatever else runs on the GPU;
//   kv_copy_kernel            256 threads x 4 x 16-byte vector loads/stores per 16 KiB piece on a
//       persistent grid (selected with CASCADE_COPY_BULK_HOST=0 / CASCADE_COPY_BULK_DEV=0).
#include <stdlib.h>
#include <string.h>

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
    int pieces_per_chunk;     // vector kernel only
    int ring_bytes;           // ring kernel: shared memory of the ring
    int piece_fixed;          // ring kernel: >0 forces this piece size (bytes), 0 = pick per call
    int ahead_sub;            // ring kernel: loads in flight ahead of the store = ring slots minus this (1 or 2)
    int record_iota;          // ring kernel: the record id of list entry i is i itself (staging buffer filled in list order)
    const int32_t *iota_check;    // with record_iota: entry i is skipped unless 0 <= iota_check[i] < iota_check_blocks
    long long iota_check_blocks;  // (the id its staging slot was, or will be, copied from / to by the copy engines)
    // fused move only
    const int32_t *dep;       // per restore: evict-list index of the entry that frees its HBM block, or -1
    int32_t *done;            // per evict entry: 16-byte units of the block already read out of HBM
    int32_t *skipped;         // per restore: pieces that were NOT written (0 = the block is complete)
    int stall;                // test hooks, see cascade_ctx::test_move_stall
    unsigned *ticket;         // ring kernel: [0] pieces handed out beyond the first one of every CTA, [1] CTAs that are
                              // done (both zero between launches: the last CTA out resets them); NULL = fixed stride
};

enum { kRoleRestore = 0, kRoleEvict = 1, kRoleMoveEvict = 2, kRoleMoveRestore = 3 };
constexpr long long kWaitCycles = 4000000000LL;  // about two seconds at 1.9 GHz

__device__ __forceinline__ int clamp_count(const int32_t *dev, int maxv) {
    if (!dev) return maxv;
    const int c = __ldcg(dev);
    return c < 0 ? 0 : (c < maxv ? c : maxv);
}

// Vector variant.  The roles are those of the ring kernel below: the two plain copies and the two grids of
// the fused evict + restore (see cascade_kv_move for how the two grids are ordered).
template <int kRole>
__global__ void __launch_bounds__(kThreads) kv_copy_kernel(const __grid_constant__ CopyArgs a) {
    constexpr bool kRestore = kRole == kRoleRestore || kRole == kRoleMoveRestore;
    __shared__ int s_skip;
    if (kRole != kRoleMoveRestore) cascade_grid_wait();
    if (kRole == kRoleMoveEvict) cascade_grid_trigger();
    const int count = clamp_count(a.n_dev, a.n_max);
    const long long per_block = (long long)a.n_chunks * a.pieces_per_chunk;
    const long long items = (long long)count * per_block;
    const long long bb = (long long)a.n_chunks * a.chunk_bytes;
    const long long limit = a.stall ? kWaitCycles / 20 : kWaitCycles;
    const int tid = threadIdx.x;
    uint32_t st = 0;
    for (long long it = blockIdx.x; it < items; it += gridDim.x) {
        long long i = it / per_block;
        const int rem = (int)(it - i * per_block);
        if (kRole == kRoleMoveEvict) i = count - 1 - i;  // blocks freed last are handed out first: read them out first
        const int c = rem / a.pieces_per_chunk;
        const int pc = rem - c * a.pieces_per_chunk;
        const long long s = __ldcg(a.src_ids + i), d = __ldcg(a.dst_ids + i);
        const long long rec_id = kRestore ? s : d, pg_id = kRestore ? d : s;
        const long long left = a.chunk_bytes - (long long)pc * kPiece;
        const int piece_bytes = (int)(left < kPiece ? left : kPiece);
        if (rec_id < 0 || rec_id >= a.record_blocks || pg_id < 0 || pg_id >= a.paged_blocks) {
            st |= CASCADE_ST_EBOUNDS;  // id outside its pool: this pair is skipped
            if (tid == 0) {
                // a skipped evict piece still counts as read, or a restore into that block would wait for nothing
                if (kRole == kRoleMoveEvict) atomicAdd(&a.done[i], piece_bytes >> 4);
                if (kRole == kRoleMoveRestore) atomicAdd(&a.skipped[i], 1);
            }
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
        if (kRole == kRoleMoveRestore) {
            const int dep = __ldcg(a.dep + i);  // the same for every thread of the CTA
            if (dep >= 0) {
                // the HBM block is being evicted by this same call: write only after it has been read out
                if (tid == 0) {
                    const volatile int32_t *flag = a.done + dep;
                    int skip = (st & CASCADE_ST_ETIMEOUT) ? 1 : 0;  // one expired wait is enough: do not queue up more
                    const long long t0 = clock64();
                    while (!skip && *flag < (int)(bb >> 4))
                        if (clock64() - t0 > limit) skip = 1;
                    if (skip) {
                        st |= CASCADE_ST_ETIMEOUT;
                        atomicAdd(&a.skipped[i], 1);
                    }
                    __threadfence();
                    s_skip = skip;
                }
                __syncthreads();
                const bool skip = s_skip != 0;
                __syncthreads();
                if (skip) continue;
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const long long off = base + (long long)u * kThreads * 16;
            if (off < a.chunk_bytes) __stcs(reinterpret_cast<uint4 *>(dst + off), v[u]);
        }
        if (kRole == kRoleMoveEvict) {
            // every thread's loads have returned once its stores are issued: this piece has left HBM; counted in
            // 16-byte units, because the two grids may cut their blocks into pieces of different sizes
            __syncthreads();
            if (tid == 0 && a.stall != 1) {
                __threadfence();
                atomicAdd(&a.done[i], piece_bytes >> 4);
            }
        }
    }
    if (st && tid == 0) atomicOr(a.status, st);
    // completion of the restore grid must imply completion of the evict grid it ran beside
    if (kRole == kRoleMoveRestore) cascade_grid_wait();
}


// ---- ring kernel: TMA bulk copies (cp.async.bulk) through a shared-memory ring ----------------------
// One elected thread per CTA moves pieces: global -> shared with an mbarrier that counts the arriving
// bytes, then shared -> global as a bulk store group.  The ring has S = ring_bytes / piece slots.  S - 1
// loads are issued before the first wait (short calls live off this); afterwards S - 2 loads are kept in
// flight ahead of the piece being stored, so that the slot refilled next was last read by the store issued
// one step EARLIER, which has long finished reading shared memory (with S - 1 in flight the refill would
// wait for the store just issued: measured 6.2 instead of 6.55 TB/s through the staging buffer).  Every
// wait is bounded: when the clock limit is hit the CTA records CASCADE_ST_ETIMEOUT, issues nothing more,
// waits (bounded again) for the loads it still has in flight, drains its store groups and returns.
//
// The same loop serves four roles:
//   kRoleRestore / kRoleEvict          the two plain copies;
//   kRoleMoveEvict / kRoleMoveRestore  the two grids of the fused evict + restore (see cascade_kv_move).
constexpr int kPieceMax = 32 * 1024;
constexpr int kPieceMin = 8 * 1024;
constexpr int kMaxStages = 16;
constexpr int kRingHost = 128 * 1024;   // at most one CTA per SM
constexpr int kRingDev = 96 * 1024;     // two CTAs per SM fit

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
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity, long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > limit) return false;
    return true;
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

template <int kRole>
__global__ void __launch_bounds__(32) kv_ring_kernel(const __grid_constant__ CopyArgs a) {
    constexpr bool kRestore = kRole == kRoleRestore || kRole == kRoleMoveRestore;
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) unsigned long long bars[kMaxStages];
    // barrier set-up touches no global memory, so it runs ahead of the wait for the preceding grid
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) mbar_init(smem_addr(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // The restore grid of the fused move is launched as a programmatic dependent of the evict grid
    // and must run BESIDE it, so it does not wait here but at its very end (see cascade_kv_move).
    if (kRole != kRoleMoveRestore) cascade_grid_wait();
    if (kRole == kRoleMoveEvict) cascade_grid_trigger();
    if (threadIdx.x != 0) {
        if (kRole == kRoleMoveRestore) cascade_grid_wait();
        return;
    }

    const int count = clamp_count(a.n_dev, a.n_max);
    // piece size: the largest of 32 / 16 / 8 KiB that still gives every CTA of the grid two pieces
    int piece = kPieceMax;
    if (a.piece_fixed > 0) {
        piece = a.piece_fixed;
    } else {
        while (piece > kPieceMin &&
               (long long)count * a.n_chunks * ((a.chunk_bytes + piece - 1) / piece) < 2LL * gridDim.x)
            piece >>= 1;
    }
    int S = a.ring_bytes / piece;
    S = S > kMaxStages ? kMaxStages : S;
    const int prime = S - 1;   // loads issued before the first wait
    const int ppc = (int)((a.chunk_bytes + piece - 1) / piece);
    const long long per_block = (long long)a.n_chunks * ppc;
    const long long items = (long long)count * per_block;
    const long long bb = (long long)a.n_chunks * a.chunk_bytes;
    const long long limit = a.stall ? kWaitCycles / 20 : kWaitCycles;
    // loads in flight ahead of the store after the first wait: a call of a few pieces per CTA is over before the
    // ring reaches a steady state and keeps every slot busy; a long one leaves the slot of the store just issued alone
    const int steady = (items < 16LL * gridDim.x || S - a.ahead_sub < 1) ? S - 1 : S - a.ahead_sub;
    uint32_t st = 0;

    long long next = blockIdx.x;  // next item of this CTA to load
    char *dst_of[kMaxStages];
    unsigned bytes_of[kMaxStages];
    int entry_of[kMaxStages];     // list index of the piece in the slot
    long long issued = 0, stored = 0;
    int claims = 0;               // pieces this CTA has taken so far
    // on demand only where it pays: calls of many pieces per CTA, pieces large enough to hide the counter's round trip
    // (measured: the fused move of 256 + 256 blocks 71 -> 76 GB/s, 64 staged blocks 5.7 -> 6.1 TB/s; calls of a few
    // pieces per CTA and 4 KiB pieces lose a few per cent)
    const bool on_demand = a.ticket != nullptr && items >= 16LL * gridDim.x && piece >= 16 * 1024;
    auto issue_next = [&]() -> bool {  // loads the next valid item into ring slot issued % S
        while (next < items) {
            const long long it = next;
            // The pieces a CTA loads before its first wait come by a fixed stride (a short call is spread evenly
            // whichever CTA starts first); the following ones are handed out on demand, so that a CTA on a slower path
            // to memory takes fewer and all of them finish together (a fixed stride leaves the last round to the CTAs
            // that happen to hold one piece more).  The counter's value is needed at the NEXT call only: its latency
            // hides behind the copy just issued.
            ++claims;
            next = (on_demand && claims >= prime) ? (long long)prime * gridDim.x + atomicAdd(a.ticket, 1u)
                                                  : next + gridDim.x;
            long long i = it / per_block;
            const int rem = (int)(it - i * per_block);
            if (kRole == kRoleMoveEvict) i = count - 1 - i;  // blocks freed last are handed out first: read them out first
            const int c = rem / ppc, pc = rem - c * ppc;
            long long s, d;
            if (a.record_iota) {   // only the paged side has a list
                s = kRestore ? i : __ldcg(a.src_ids + i);
                d = kRestore ? __ldcg(a.dst_ids + i) : i;
                if (a.iota_check) {
                    const long long far = __ldcg(a.iota_check + i);
                    if (far < 0 || far >= a.iota_check_blocks) { if (kRestore) s = -1; else d = -1; }
                }
            } else {
                s = __ldcg(a.src_ids + i);
                d = __ldcg(a.dst_ids + i);
            }
            const long long rec_id = kRestore ? s : d, pg_id = kRestore ? d : s;
            const long long off = (long long)pc * piece;
            const long long left = a.chunk_bytes - off;
            const unsigned bytes = (unsigned)(left < piece ? left : piece);
            if (rec_id < 0 || rec_id >= a.record_blocks || pg_id < 0 || pg_id >= a.paged_blocks) {
                st |= CASCADE_ST_EBOUNDS;  // id outside its pool: this pair is skipped
                // a skipped evict piece still counts as read, or a restore into that block would wait for nothing
                if (kRole == kRoleMoveEvict) atomicAdd(&a.done[i], (int)(bytes >> 4));
                if (kRole == kRoleMoveRestore) atomicAdd(&a.skipped[i], 1);
                continue;
            }
            char *rec = a.record + rec_id * bb + (long long)c * a.chunk_bytes + off;
            char *pg = a.paged + (long long)c * a.chunk_stride + pg_id * a.block_stride + off;
            const int slot = (int)(issued % S);
            const unsigned bar = smem_addr(&bars[slot]);
            // test hook 2: the very first piece of CTA 0 announces more bytes than it loads, so its wait runs out
            const bool short_load = a.stall == 2 && blockIdx.x == 0 && issued == 0;
            mbar_expect_tx(bar, bytes + (short_load ? 16u : 0u));
            bulk_load(smem_addr(ring + (size_t)slot * piece), kRestore ? rec : pg, bytes, bar);
            dst_of[slot] = kRestore ? pg : rec;
            bytes_of[slot] = bytes;
            entry_of[slot] = (int)i;
            ++issued;
            return true;
        }
        return false;
    };
    for (int k = 0; k < prime; ++k)
        if (!issue_next()) break;
    while (stored < issued) {
        const int slot = (int)(stored % S);
        const unsigned parity = (unsigned)((stored / S) & 1);
        if (!mbar_wait_bounded(smem_addr(&bars[slot]), parity, limit)) {
            // give up: record it, issue nothing more, but do not leave while loads still target this CTA's ring
            st |= CASCADE_ST_ETIMEOUT;
            const long long t_giveup = clock64();   // one more limit for all of them together, not one each
            for (long long q = stored + 1; q < issued; ++q) {
                const long long left = limit - (clock64() - t_giveup);
                mbar_wait_bounded(smem_addr(&bars[q % S]), (unsigned)((q / S) & 1), left > 0 ? left : 0);
            }
            if (kRole == kRoleMoveRestore)
                for (long long q = stored; q < issued; ++q) atomicAdd(&a.skipped[entry_of[q % S]], 1);
            break;
        }
        bool skip = false;
        if (kRole == kRoleMoveEvict) {
            // this piece of the block has left HBM; counted in 16-byte units, because the two grids may
            // cut their blocks into pieces of different sizes
            if (a.stall != 1) atomicAdd(&a.done[entry_of[slot]], (int)(bytes_of[slot] >> 4));
        } else if (kRole == kRoleMoveRestore) {
            const int dep = __ldcg(a.dep + entry_of[slot]);
            if (dep >= 0) {
                // the HBM block is being evicted by this same call: write only after it has been read out
                const volatile int32_t *flag = a.done + dep;
                const long long t0 = clock64();
                if (st & CASCADE_ST_ETIMEOUT) skip = true;  // one expired wait is enough: do not queue up more
                while (!skip && *flag < (int)(bb >> 4)) {
                    if (clock64() - t0 > limit) {
                        st |= CASCADE_ST_ETIMEOUT;
                        skip = true;
                    }
                }
                __threadfence();
                if (skip) atomicAdd(&a.skipped[entry_of[slot]], 1);
            }
        }
        if (!skip) bulk_store(dst_of[slot], smem_addr(ring + (size_t)slot * piece), bytes_of[slot]);
        ++stored;
        // every store but the one just issued has finished reading shared memory
        asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        if (issued - stored < steady) issue_next();
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (st) atomicOr(a.status, st);
    // The last CTA out leaves the two counters at zero for the next launch that uses them.  Every CTA has made its last
    // claim by then: the test of `next` waits for the value of this CTA's last claim (also on the give-up path, where
    // nothing else reads it), and the fences keep the claim, the count of CTAs that are done and the reset in this order.
    if (on_demand && next >= 0) {
        __threadfence();
        if (atomicAdd(a.ticket + 1, 1u) == gridDim.x - 1) {
            __threadfence();
            a.ticket[0] = 0;
            a.ticket[1] = 0;
        }
    }
    // completion of this grid must imply completion of the evict grid it ran beside
    if (kRole == kRoleMoveRestore) cascade_grid_wait();
}

// ---- fused evict + restore ("move"): both directions of the host link at once ----------------------
// Three launches on the caller's stream:
//   1. kv_move_prepare_kernel (one CTA): zeroes the per-entry counters and finds, for every restore, the
//      evict entry that frees its HBM block (the tier plan hands freed blocks out again at once) through an
//      open-addressing hash table over the evicted block ids: linear work in the two list lengths;
//   2. the evict grid (role kRoleMoveEvict), a little under half of the SMs: device -> host; after every piece that has
//      left HBM it bumps that entry's counter.  It signals "dependents may launch" as its first action;
//   3. the restore grid (role kRoleMoveRestore), on the other half, launched as a PROGRAMMATIC DEPENDENT of
//      grid 2: the hardware starts it only once every CTA of the evict grid is running (or done), so a
//      restore CTA that waits for a counter always waits for a CTA that is already on an SM and never waits
//      itself: no deadlock however busy the GPU is with other work.  A restore into a block that the same
//      call evicts stores only after that block's counter says it has been read out completely.
// Without programmatic launch (CASCADE_PDL=0) grid 3 simply starts after grid 2 has finished.
// Measured on B200: when both grids use the bulk-copy ring, the restore grid's bulk reads of host memory make
// no progress until the evict grid's bulk writes are over (52 GB/s, the two directions one after the other);
// with the restore grid on plain vector loads both directions run at once (71 - 80 GB/s), so by default the
// evict grid is the ring kernel and the restore grid the vector kernel (CASCADE_MOVE_VECTOR, bit 0 = restore
// grid, bit 1 = evict grid on the vector kernel).
struct PrepareArgs {
    const int32_t *evict_src, *restore_dst;
    const int32_t *n_evict_dev, *n_restore_dev;
    int n_evict_max, n_restore_max;
    int32_t *skipped, *dep, *done, *hkeys, *hvals;
    int hash_cap;  // power of two
};

// multiplicative hashing: the HIGH bits of the product depend on every bit of the id (block ids that are all multiples
// of a power of two would share the low ones)
__device__ __forceinline__ unsigned hash_id(int32_t g, int bits) { return ((unsigned)g * 2654435761u) >> (32 - bits); }

__global__ void __launch_bounds__(1024) kv_move_prepare_kernel(const __grid_constant__ PrepareArgs a) {
    cascade_grid_wait();
    cascade_grid_trigger();
    const int ne = clamp_count(a.n_evict_dev, a.n_evict_max), nr = clamp_count(a.n_restore_dev, a.n_restore_max);
    const int tid = threadIdx.x, T = blockDim.x;
    int H = 64, hbits = 6;  // table size: at most half full
    while (H < 2 * ne && H < a.hash_cap) { H <<= 1; ++hbits; }
    const unsigned mask = (unsigned)H - 1u;
    for (int h = tid; h < H; h += T) {
        a.hkeys[h] = -1;
        a.hvals[h] = -1;
    }
    for (int j = tid; j < ne; j += T) a.done[j] = 0;
    for (int r = tid; r < nr; r += T) a.skipped[r] = 0;
    __syncthreads();
    for (int j = tid; j < ne; j += T) {
        const int32_t g = a.evict_src[j];
        if (g < 0) continue;  // never matches a valid destination
        unsigned h = hash_id(g, hbits);
        for (int probe = 0; probe < H; ++probe) {
            const int32_t prev = atomicCAS(&a.hkeys[h], -1, g);
            if (prev == -1 || prev == g) {
                atomicMax(&a.hvals[h], j);  // the LAST entry that evicts the block is the one to wait for
                break;
            }
            h = (h + 1) & mask;
        }
    }
    __syncthreads();
    for (int r = tid; r < nr; r += T) {
        const int32_t g = a.restore_dst[r];
        int dep = -1;
        if (g >= 0) {
            unsigned h = hash_id(g, hbits);
            for (int probe = 0; probe < H; ++probe) {
                const int32_t k = a.hkeys[h];
                if (k == g) { dep = a.hvals[h]; break; }
                if (k == -1) break;
                h = (h + 1) & mask;
            }
        }
        a.dep[r] = dep;
    }
}

constexpr int kMaxMoveList = 1 << 28;   // longest list the fused move accepts (the hash table has twice as many slots)

int hash_capacity(int n_evict_max) {
    int H = 64;
    while (H < 2 * (long long)n_evict_max && H < (1 << 30)) H <<= 1;
    return H;
}

int check_layout(const cascade_kv_layout *l, const void *paged, const void *record, long long record_blocks) {
    if (!l || !paged || !record) return CASCADE_EINVAL;
    if (l->n_blocks < 0 || record_blocks < 0 || l->n_chunks < 1 || l->chunk_bytes < 16) return CASCADE_EINVAL;
    if ((l->chunk_bytes | l->chunk_stride | l->block_stride) & 15) return CASCADE_EINVAL;
    if (l->chunk_stride < 0 || l->block_stride < 0) return CASCADE_EINVAL;
    if (((uintptr_t)paged | (uintptr_t)record) & 15) return CASCADE_EINVAL;
    return CASCADE_OK;
}

void fill_copy_args(CopyArgs &a, const cascade_ctx *ctx, const cascade_kv_layout *l, char *paged, char *record,
                    long long record_blocks, const int32_t *src_ids, const int32_t *dst_ids, const int32_t *n_dev,
                    int n_max) {
    a = CopyArgs{};
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
    a.piece_fixed = ctx->copy_piece;
    a.ahead_sub = ctx->copy_ahead_sub;
    a.stall = ctx->test_move_stall;
}

// Work counters of one ring launch: a pair out of a small pool, taken in turn, so that two launches that overlap (the
// two grids of the fused move; launches a caller put on two streams against the rule) never share one.  A pair is
// zero whenever no launch is using it: the last CTA out resets it.
constexpr int kTicketPairs = 64;

unsigned *next_ticket(cascade_ctx *ctx) {
    if (!ctx->copy_dynamic) return nullptr;
    return ctx->copy_tickets + 2 * (ctx->copy_ticket_seq++ % kTicketPairs);
}

// the ring kernels need more dynamic shared memory than the default limit: opt in once per device
template <int kRole>
cudaError_t configure_ring(int device) {
    static CascadeDeviceOnce configured;
    if (configured.is_set(device)) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kv_ring_kernel<kRole>, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingHost);
    if (e == cudaSuccess) configured.set(device);
    return e;
}

template <bool kRestore>
int launch_copy(cascade_ctx *ctx, const cascade_kv_layout *l, char *paged, char *record, long long record_blocks,
                int record_is_device, const int32_t *src_ids, const int32_t *dst_ids, const int32_t *n_dev, int n_max,
                cudaStream_t s) {
    if (!ctx || n_max < 0) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (n_max == 0) return CASCADE_OK;
    int rc = check_layout(l, paged, record, record_blocks);
    if (rc != CASCADE_OK) return rc;
    if (!src_ids || !dst_ids) return CASCADE_EINVAL;
    CopyArgs a;
    fill_copy_args(a, ctx, l, paged, record, record_blocks, src_ids, dst_ids, n_dev, n_max);
    const int mode = record_is_device ? ctx->copy_bulk_dev : ctx->copy_bulk_host;
    if (mode) {
        // TMA ring: one elected thread per CTA; `mode` CTAs per SM
        a.ring_bytes = mode > 1 ? kRingDev : kRingHost;
        if (ctx->copy_ring_kb > 0) a.ring_bytes = ctx->copy_ring_kb * 1024;
        const long long items = (long long)n_max * l->n_chunks * ((l->chunk_bytes + kPieceMin - 1) / kPieceMin);
        long long grid = (long long)ctx->num_sms * (mode > 1 ? mode : 1);
        // Over the host link the rate does not depend on the grid between 40 and 148 CTAs (evict 52.7 GB/s with 24, 65 or
        // 148; restore 50.1 / 51.4 / 50.6 GB/s; one block and sixteen blocks take the same time too), so the copy takes
        // 44 % of the SMs and leaves the shared memory of the others to whatever else runs on the GPU.
        if (!record_is_device)
            grid = ctx->copy_grid_host > 0 ? ctx->copy_grid_host : (ctx->num_sms * 44 + 50) / 100;
        if (grid < 1) grid = 1;
        if (grid > items) grid = items;
        constexpr int role = kRestore ? kRoleRestore : kRoleEvict;
        a.ticket = next_ticket(ctx);
        CASCADE_CUDA_TRY(ctx, configure_ring<role>(ctx->device));
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)grid), dim3(32), (size_t)a.ring_bytes, s,
                                             kv_ring_kernel<role>, a));
        return CASCADE_OK;
    }
    a.pieces_per_chunk = (int)((l->chunk_bytes + kPiece - 1) / kPiece);
    const long long items = (long long)n_max * l->n_chunks * a.pieces_per_chunk;
    const int per_sm = record_is_device ? ctx->copy_ctas_dev : ctx->copy_ctas_host;
    long long grid = (long long)ctx->num_sms * per_sm;
    if (grid > items) grid = items;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)grid), dim3(kThreads), 0, s,
                                         kv_copy_kernel<kRestore ? kRoleRestore : kRoleEvict>, a));
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

extern "C" int64_t cascade_kv_move_scratch_len(int n_evict_max, int n_restore_max) {
    if (n_evict_max < 0 || n_restore_max < 0 || n_evict_max > kMaxMoveList || n_restore_max > kMaxMoveList) return -1;
    return 2 * (int64_t)n_restore_max + (int64_t)n_evict_max + 2 * (int64_t)hash_capacity(n_evict_max);
}

extern "C" int cascade_kv_move(cascade_ctx *ctx, const cascade_kv_layout *hbm, void *hbm_pool, void *host_pool,
                               int64_t host_blocks, const int32_t *evict_src, const int32_t *evict_dst,
                               const int32_t *n_evict_dev, int n_evict_max, const int32_t *restore_src,
                               const int32_t *restore_dst, const int32_t *n_restore_dev, int n_restore_max,
                               int32_t *scratch, void *stream) {
    CascadeRange nvtx_range("cascade_kv_move");
    if (!ctx || n_evict_max < 0 || n_restore_max < 0) return CASCADE_EINVAL;
    if (n_evict_max > kMaxMoveList || n_restore_max > kMaxMoveList) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (n_evict_max == 0 && n_restore_max == 0) return CASCADE_OK;
    int rc = check_layout(hbm, hbm_pool, host_pool, host_blocks);
    if (rc != CASCADE_OK) return rc;
    if (!scratch || (n_evict_max > 0 && (!evict_src || !evict_dst)) || (n_restore_max > 0 && (!restore_src || !restore_dst)))
        return CASCADE_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    // scratch: skipped[n_restore_max] | dep[n_restore_max] | done[n_evict_max] | hash keys | hash values
    PrepareArgs p;
    p.evict_src = evict_src;
    p.restore_dst = restore_dst;
    p.n_evict_dev = n_evict_dev;
    p.n_restore_dev = n_restore_dev;
    p.n_evict_max = n_evict_max;
    p.n_restore_max = n_restore_max;
    p.hash_cap = hash_capacity(n_evict_max);
    p.skipped = scratch;
    p.dep = p.skipped + n_restore_max;
    p.done = p.dep + n_restore_max;
    p.hkeys = p.done + n_evict_max;
    p.hvals = p.hkeys + p.hash_cap;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(1), dim3(1024), 0, s, kv_move_prepare_kernel, p));

    const long long ppc_max = (hbm->chunk_bytes + kPieceMin - 1) / kPieceMin;
    // SMs per grid: a little under half of them.  Measured on B200 (148 SMs), 512 + 512 blocks of 2 MiB: 65 + 65 gives
    // 79 GB/s, 74 + 74 gives 77, 58 + 58 gives 78, 50 + 50 gives 75: with fewer posted writes queued towards the host the
    // restore grid's read requests get through sooner.
    int half = (ctx->num_sms * 44 + 50) / 100;
    if (ctx->move_ctas > 0 && ctx->move_ctas <= ctx->num_sms / 2) half = ctx->move_ctas;
    if (half < 1) half = 1;
    int half_r = half;
    if (ctx->move_ctas_restore > 0 && ctx->move_ctas_restore <= ctx->num_sms / 2) half_r = ctx->move_ctas_restore;
    CASCADE_CUDA_TRY(ctx, configure_ring<kRoleMoveEvict>(ctx->device));
    CASCADE_CUDA_TRY(ctx, configure_ring<kRoleMoveRestore>(ctx->device));
    CopyArgs e, r;
    fill_copy_args(e, ctx, hbm, (char *)hbm_pool, (char *)host_pool, host_blocks, evict_src, evict_dst, n_evict_dev,
                   n_evict_max);
    fill_copy_args(r, ctx, hbm, (char *)hbm_pool, (char *)host_pool, host_blocks, restore_src, restore_dst,
                   n_restore_dev, n_restore_max);
    e.ring_bytes = r.ring_bytes = ctx->copy_ring_kb > 0 ? ctx->copy_ring_kb * 1024 : kRingHost;
    e.ticket = next_ticket(ctx);
    r.ticket = next_ticket(ctx);
    e.done = r.done = p.done;
    e.dep = r.dep = p.dep;
    e.skipped = r.skipped = p.skipped;
    // the evict grid is launched even when its list is empty: the restore grid is ordered behind it
    long long ge = half, gr = half_r;
    const long long items_e = (long long)n_evict_max * hbm->n_chunks * ppc_max;
    const long long items_r = (long long)n_restore_max * hbm->n_chunks * ppc_max;
    if (ge > items_e) ge = items_e < 1 ? 1 : items_e;
    if (gr > items_r) gr = items_r;
    e.pieces_per_chunk = r.pieces_per_chunk = (int)((hbm->chunk_bytes + kPiece - 1) / kPiece);
    const int vec_per_sm = ctx->copy_ctas_host;
    if (ctx->move_vector & 2) {
        long long g = (long long)half * vec_per_sm;
        const long long iv = (long long)n_evict_max * hbm->n_chunks * e.pieces_per_chunk;
        if (g > iv) g = iv < 1 ? 1 : iv;
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)g), dim3(kThreads), 0, s,
                                             kv_copy_kernel<kRoleMoveEvict>, e));
    } else {
        CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)ge), dim3(32), (size_t)e.ring_bytes, s,
                                             kv_ring_kernel<kRoleMoveEvict>, e));
    }
    if (gr > 0) {
        if (ctx->move_vector & 1) {
            long long g = (long long)half_r * vec_per_sm;
            const long long iv = (long long)n_restore_max * hbm->n_chunks * r.pieces_per_chunk;
            if (g > iv) g = iv;
            CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)g), dim3(kThreads), 0, s,
                                                 kv_copy_kernel<kRoleMoveRestore>, r));
        } else {
            CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3((unsigned)gr), dim3(32), (size_t)r.ring_bytes, s,
                                                 kv_ring_kernel<kRoleMoveRestore>, r));
        }
    }
    return CASCADE_OK;
}


// ---- evict + restore through the copy engines -------------------------------------------------------
// The lists live in device memory, the copy engines are driven by the host: a small kernel publishes
// the two counts and the lists' live entries into a pinned mailbox, the host waits for it ONCE, then
//   evictions: [stream] gather the paged blocks into the staging buffer (ring kernel, HBM to HBM)
//              [side 1] one cudaMemcpyAsync per run of consecutive host records, staging -> host pool
//   restores:  [side 0] one cudaMemcpyAsync per run of consecutive host records, host pool -> staging
//              [stream] scatter the staged blocks into the paged pool (ring kernel, HBM to HBM)
// with every gather ahead of every scatter on the caller's stream (a freed block may be handed out again
// at once) and the two side streams running beside each other, so both directions of the link are busy.
// Gathers and fills go in batches (a small first one) so that the link starts after microseconds.
namespace {

struct PublishArgs {
    const int32_t *evict_src, *evict_dst, *restore_src, *restore_dst;
    const int32_t *n_evict_dev, *n_restore_dev;
    int n_evict_max, n_restore_max;
    int32_t *mailbox;   // pinned, mapped host memory
};

__global__ void __launch_bounds__(256) kv_publish_lists_kernel(const __grid_constant__ PublishArgs a) {
    cascade_grid_wait();
    const int ne = clamp_count(a.n_evict_dev, a.n_evict_max), nr = clamp_count(a.n_restore_dev, a.n_restore_max);
    const int i = blockIdx.x * blockDim.x + threadIdx.x, stride = gridDim.x * blockDim.x;
    int32_t *es = a.mailbox + 2, *ed = es + a.n_evict_max, *rs = ed + a.n_evict_max, *rd = rs + a.n_restore_max;
    for (int j = i; j < ne; j += stride) {
        es[j] = a.evict_src[j];
        ed[j] = a.evict_dst[j];
    }
    for (int j = i; j < nr; j += stride) {
        rs[j] = a.restore_src[j];
        rd[j] = a.restore_dst[j];
    }
    if (i == 0) {
        a.mailbox[0] = ne;
        a.mailbox[1] = nr;
    }
}

constexpr int kFirstBatch = 8;    // blocks in the first gather / fill batch: the link starts early
constexpr int kBatch = 64;

// one HBM-to-HBM pass of the ring kernel between the paged pool and a staging region filled in list order
template <bool kRestore>
int launch_staged_pass(cascade_ctx *ctx, const cascade_kv_layout *l, char *paged, char *region, const int32_t *paged_ids,
                       const int32_t *host_ids, long long host_blocks, int m, cudaStream_t s) {
    CopyArgs a;
    fill_copy_args(a, ctx, l, paged, region, m, kRestore ? nullptr : paged_ids, kRestore ? paged_ids : nullptr, nullptr, m);
    a.record_iota = 1;
    a.iota_check = host_ids;
    a.iota_check_blocks = host_blocks;
    a.ring_bytes = ctx->copy_ring_kb > 0 ? ctx->copy_ring_kb * 1024 : kRingDev;
    const long long items = (long long)m * l->n_chunks * ((l->chunk_bytes + kPieceMin - 1) / kPieceMin);
    long long grid = (long long)ctx->num_sms * 2;
    if (grid > items) grid = items;
    constexpr int role = kRestore ? kRoleRestore : kRoleEvict;
    a.ticket = next_ticket(ctx);
    CASCADE_CUDA_TRY(ctx, configure_ring<role>(ctx->device));
    CASCADE_CUDA_TRY(ctx, cascade_launch(false, 0, dim3((unsigned)grid), dim3(32), (size_t)a.ring_bytes, s,
                                         kv_ring_kernel<role>, a));
    return CASCADE_OK;
}

}  // namespace

extern "C" int64_t cascade_kv_mailbox_len(int n_evict_max, int n_restore_max) {
    if (n_evict_max < 0 || n_restore_max < 0) return -1;
    return 2 + 2 * (int64_t)n_evict_max + 2 * (int64_t)n_restore_max;
}

extern "C" int cascade_kv_move_staged(cascade_ctx *ctx, const cascade_kv_layout *hbm, void *hbm_pool, void *host_pool,
                                      int64_t host_blocks, const int32_t *evict_src, const int32_t *evict_dst,
                                      const int32_t *n_evict_dev, int n_evict_max, const int32_t *restore_src,
                                      const int32_t *restore_dst, const int32_t *n_restore_dev, int n_restore_max,
                                      void *staging, int64_t staging_blocks, int32_t *mailbox, void *stream) {
    CascadeRange nvtx_range("cascade_kv_move_staged");
    if (!ctx || n_evict_max < 0 || n_restore_max < 0) return CASCADE_EINVAL;
    if (!cascade_on_ctx_device(ctx)) return CASCADE_EINVAL;
    if (n_evict_max == 0 && n_restore_max == 0) return CASCADE_OK;
    int rc = check_layout(hbm, hbm_pool, host_pool, host_blocks);
    if (rc != CASCADE_OK) return rc;
    if (!staging || !mailbox || staging_blocks < 1 || ((uintptr_t)staging & 15)) return CASCADE_EINVAL;
    if ((n_evict_max > 0 && (!evict_src || !evict_dst)) || (n_restore_max > 0 && (!restore_src || !restore_dst)))
        return CASCADE_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    cudaStream_t *s_fill = ctx->ce_stream, *s_drain = ctx->ce_stream + 2;
    cudaEvent_t ev_lists = ctx->ce_event[0], ev_gather = ctx->ce_event[1], ev_scatter = ctx->ce_event[2];
    cudaEvent_t *ev_fill = ctx->ce_event + 3, *ev_drain = ctx->ce_event + 5;
    const int L = ctx->ce_lanes;   // copies of one direction alternate between L side streams: the engines' per-copy
                                   // set-up of one stream hides behind the transfer of the other
    const long long bb = (long long)hbm->n_chunks * hbm->chunk_bytes;

    // 1. lists -> pinned mailbox, and the one host wait of the call
    PublishArgs p = {evict_src, evict_dst, restore_src, restore_dst, n_evict_dev, n_restore_dev, n_evict_max, n_restore_max, mailbox};
    const int most = n_evict_max > n_restore_max ? n_evict_max : n_restore_max;
    int pgrid = (most + 255) / 256;
    if (pgrid > ctx->num_sms) pgrid = ctx->num_sms;
    CASCADE_CUDA_TRY(ctx, cascade_launch(ctx->pdl, 0, dim3(pgrid), dim3(256), 0, s, kv_publish_lists_kernel, p));
    CASCADE_CUDA_TRY(ctx, cudaEventRecord(ev_lists, s));
    CASCADE_CUDA_TRY(ctx, cudaEventSynchronize(ev_lists));
    const int ne = mailbox[0], nr = mailbox[1];
    if (ne < 0 || ne > n_evict_max || nr < 0 || nr > n_restore_max) return CASCADE_EINVAL;
    if (ne > 0 && nr > 0 && staging_blocks < 2) return CASCADE_EINVAL;   // one block of staging per direction at least
    const int32_t *h_es = mailbox + 2, *h_ed = h_es + n_evict_max, *h_rs = h_ed + n_evict_max, *h_rd = h_rs + n_restore_max;
    const long long paged_blocks = hbm->n_blocks;

    // 2. does a restore read a host record that this call's evictions write?  Then the fills wait for the drains.
    bool fill_after_drain = false;
    if (ne > 0 && nr > 0) {
        const size_t words = (size_t)(host_blocks + 63) / 64;
        if (words > ctx->ce_bitmap_words) {
            unsigned long long *nb = (unsigned long long *)realloc(ctx->ce_bitmap, words * sizeof(unsigned long long));
            if (!nb) return CASCADE_ENOMEM;
            ctx->ce_bitmap = nb;
            ctx->ce_bitmap_words = words;
        }
        memset(ctx->ce_bitmap, 0, words * sizeof(unsigned long long));
        for (int i = 0; i < ne; ++i)
            if (h_ed[i] >= 0 && h_ed[i] < host_blocks) ctx->ce_bitmap[h_ed[i] >> 6] |= 1ull << (h_ed[i] & 63);
        for (int i = 0; i < nr && !fill_after_drain; ++i)
            if (h_rs[i] >= 0 && h_rs[i] < host_blocks && (ctx->ce_bitmap[h_rs[i] >> 6] >> (h_rs[i] & 63) & 1))
                fill_after_drain = true;
    }

    // 3. staging regions: one per direction, in proportion to the lists
    long long region_e = ne == 0 ? 0 : (nr == 0 ? staging_blocks : staging_blocks * ne / ((long long)ne + nr));
    if (ne > 0 && region_e < 1) region_e = 1;
    if (nr > 0 && region_e > staging_blocks - 1) region_e = staging_blocks - 1;
    const long long region_r = staging_blocks - region_e;
    char *stage_e = (char *)staging, *stage_r = (char *)staging + region_e * bb;

    // Helpers: one batch of drains / fills (one cudaMemcpyAsync per run of consecutive host records, pairs with an
    // id outside its pool left out; the gather / scatter kernel sets the status bit for them).
    bool drained_any = false;
    int lane_e = 0, lane_r = 0;
    auto drain_batch = [&](int off, int m, long long pos) -> int {
        for (int i = 0; i < m;) {
            const long long rec = h_ed[off + i], pg = h_es[off + i];
            if (rec < 0 || rec >= host_blocks || pg < 0 || pg >= paged_blocks) {
                i += 1;
                continue;
            }
            int run = 1;
            while (i + run < m && h_ed[off + i + run] == rec + run && rec + run < host_blocks &&
                   h_es[off + i + run] >= 0 && h_es[off + i + run] < paged_blocks)
                ++run;
            CASCADE_CUDA_TRY(ctx, cudaMemcpyAsync((char *)host_pool + rec * bb, stage_e + (pos + i) * bb,
                                                  (size_t)run * bb, cudaMemcpyDeviceToHost, s_drain[lane_e]));
            lane_e = (lane_e + 1) % L;
            i += run;
        }
        for (int k = 0; k < L; ++k) CASCADE_CUDA_TRY(ctx, cudaEventRecord(ev_drain[k], s_drain[k]));
        drained_any = true;
        return CASCADE_OK;
    };
    auto fill_batch = [&](int off, int m, long long pos) -> int {
        for (int i = 0; i < m;) {
            const long long rec = h_rs[off + i], pg = h_rd[off + i];
            if (rec < 0 || rec >= host_blocks || pg < 0 || pg >= paged_blocks) {
                i += 1;
                continue;
            }
            int run = 1;
            while (i + run < m && h_rs[off + i + run] == rec + run && rec + run < host_blocks &&
                   h_rd[off + i + run] >= 0 && h_rd[off + i + run] < paged_blocks)
                ++run;
            CASCADE_CUDA_TRY(ctx, cudaMemcpyAsync(stage_r + (pos + i) * bb, (const char *)host_pool + rec * bb,
                                                  (size_t)run * bb, cudaMemcpyHostToDevice, s_fill[lane_r]));
            lane_r = (lane_r + 1) % L;
            i += run;
        }
        return CASCADE_OK;
    };
    // the fills follow everything issued earlier on the caller's stream: an earlier call's scatter may still read the
    // staging region, an earlier kernel may still write the host records read here
    for (int k = 0; k < L; ++k) CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s_fill[k], ev_lists, 0));

    if (region_e >= ne && region_r >= nr && !fill_after_drain) {
        // 4a. Both lists fit their regions: drains and fills are queued ALTERNATELY, batch by batch, so that neither side
        // stream runs dry while the host waits for room in the other one's queue (the driver makes the host wait once a
        // stream holds about a thousand pending operations).  One scatter over all restores follows every gather.
        int off_e = 0, off_r = 0, batch = kFirstBatch;
        while (off_e < ne || off_r < nr) {
            if (off_e < ne) {
                const int m = ne - off_e < batch ? ne - off_e : batch;
                rc = launch_staged_pass<false>(ctx, hbm, (char *)hbm_pool, stage_e + (long long)off_e * bb, evict_src + off_e,
                                               evict_dst + off_e, host_blocks, m, s);
                if (rc != CASCADE_OK) return rc;
                CASCADE_CUDA_TRY(ctx, cudaEventRecord(ev_gather, s));
                for (int k = 0; k < L; ++k) CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s_drain[k], ev_gather, 0));
                rc = drain_batch(off_e, m, off_e);
                if (rc != CASCADE_OK) return rc;
                off_e += m;
            }
            if (off_r < nr) {
                // fills in step with the drains: both lists are through their queues at about the same time
                long long m = ne > 0 ? ((long long)batch * nr + ne - 1) / ne : batch;
                m = m < 1 ? 1 : (m > nr - off_r ? nr - off_r : m);
                rc = fill_batch(off_r, (int)m, off_r);
                if (rc != CASCADE_OK) return rc;
                off_r += (int)m;
            }
            batch = kBatch;
        }
        if (nr > 0) {
            for (int k = 0; k < L; ++k) {
                CASCADE_CUDA_TRY(ctx, cudaEventRecord(ev_fill[k], s_fill[k]));
                CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s, ev_fill[k], 0));
            }
            rc = launch_staged_pass<true>(ctx, hbm, (char *)hbm_pool, stage_r, restore_dst, restore_src, host_blocks, nr, s);
            if (rc != CASCADE_OK) return rc;
            CASCADE_CUDA_TRY(ctx, cudaEventRecord(ev_scatter, s));
        }
    } else {
    // 4b. A staging buffer smaller than the lists (or fills that must wait for drains): the two lists one after the
    // other in the host's program, each batch reusing its region only after the batch before has left it.
    {
        long long pos = 0;
        int batch = kFirstBatch;
        for (int off = 0; off < ne;) {
            int m = ne - off < batch ? ne - off : batch;
            if (m > region_e) m = (int)region_e;
            if (pos + m > region_e) {   // wrap: everything drained so far must have left the region
                pos = 0;
                if (drained_any)
                    for (int k = 0; k < L; ++k) CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s, ev_drain[k], 0));
            }
            rc = launch_staged_pass<false>(ctx, hbm, (char *)hbm_pool, stage_e + pos * bb, evict_src + off,
                                           evict_dst + off, host_blocks, m, s);
            if (rc != CASCADE_OK) return rc;
            CASCADE_CUDA_TRY(ctx, cudaEventRecord(ev_gather, s));
            for (int k = 0; k < L; ++k) CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s_drain[k], ev_gather, 0));
            rc = drain_batch(off, m, pos);
            if (rc != CASCADE_OK) return rc;
            pos += m;
            off += m;
            batch = kBatch;
        }
    }
    {
        for (int k = 0; k < L; ++k) {
            if (fill_after_drain && drained_any)
                for (int j = 0; j < L; ++j) CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s_fill[k], ev_drain[j], 0));
        }
        long long pos = 0;
        int batch = kFirstBatch;
        bool scattered_any = false;
        for (int off = 0; off < nr;) {
            int m = nr - off < batch ? nr - off : batch;
            if (m > region_r) m = (int)region_r;
            if (pos + m > region_r) {
                pos = 0;
                if (scattered_any)
                    for (int k = 0; k < L; ++k) CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s_fill[k], ev_scatter, 0));
            }
            rc = fill_batch(off, m, pos);
            if (rc != CASCADE_OK) return rc;
            for (int k = 0; k < L; ++k) {
                CASCADE_CUDA_TRY(ctx, cudaEventRecord(ev_fill[k], s_fill[k]));
                CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s, ev_fill[k], 0));
            }
            rc = launch_staged_pass<true>(ctx, hbm, (char *)hbm_pool, stage_r + pos * bb, restore_dst + off,
                                          restore_src + off, host_blocks, m, s);
            if (rc != CASCADE_OK) return rc;
            CASCADE_CUDA_TRY(ctx, cudaEventRecord(ev_scatter, s));
            scattered_any = true;
            pos += m;
            off += m;
            batch = kBatch;
        }
    }
    }
    // 6. completion of the caller's stream implies that every host record has been written
    if (drained_any)
        for (int k = 0; k < L; ++k) CASCADE_CUDA_TRY(ctx, cudaStreamWaitEvent(s, ev_drain[k], 0));
    return CASCADE_OK;
}
