// cascade_kv_restore / cascade_kv_evict: paged KV-block copies between a record-major pool
// (pinned host memory read or written over the host link, or a device staging buffer) and the
// paged HBM pool, driven by (src id, dst id) lists that live in device memory.
//
// The bytes are opaque.  A block is n_chunks pieces of chunk_bytes; on the record side they are
// back to back, on the HBM side chunk c of block b sits at c*chunk_stride + b*block_stride.
// Work is cut into 16 KiB pieces (one CTA iteration each: 256 threads x 4 x 16-byte vectors, all
// loads issued before the first store) and spread over a persistent grid, so a single 2 MiB block
// already occupies 128 CTAs and every access is a fully coalesced 512-byte warp transaction.
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
    a.pieces_per_chunk = (int)((l->chunk_bytes + kPiece - 1) / kPiece);
    const long long items = (long long)n_max * l->n_chunks * a.pieces_per_chunk;
    const int per_sm = record_is_device ? ctx->copy_ctas_dev : ctx->copy_ctas_host;
    long long grid = (long long)ctx->num_sms * per_sm;
    if (grid > items) grid = items;
    kv_copy_kernel<kRestore><<<(unsigned)grid, kThreads, 0, s>>>(a);
    CASCADE_CUDA_TRY(ctx, cudaGetLastError());
    return CASCADE_OK;
}

}  // namespace

extern "C" int cascade_kv_restore(cascade_ctx *ctx, const cascade_kv_layout *hbm, void *hbm_pool, const void *src_pool,
                                  int64_t src_blocks, int src_is_device, const int32_t *src_ids,
                                  const int32_t *dst_ids, const int32_t *n_copies_dev, int n_copies_max,
                                  void *stream) {
    return launch_copy<true>(ctx, hbm, (char *)hbm_pool, (char *)const_cast<void *>(src_pool), src_blocks,
                             src_is_device, src_ids, dst_ids, n_copies_dev, n_copies_max, (cudaStream_t)stream);
}

extern "C" int cascade_kv_evict(cascade_ctx *ctx, const cascade_kv_layout *hbm, const void *hbm_pool, void *dst_pool,
                                int64_t dst_blocks, int dst_is_device, const int32_t *src_ids, const int32_t *dst_ids,
                                const int32_t *n_copies_dev, int n_copies_max, void *stream) {
    return launch_copy<false>(ctx, hbm, (char *)const_cast<void *>(hbm_pool), (char *)dst_pool, dst_blocks,
                              dst_is_device, src_ids, dst_ids, n_copies_dev, n_copies_max, (cudaStream_t)stream);
}
