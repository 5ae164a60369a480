// Block-wide scans and sums over elements laid out as (warp, round, lane): K elements per thread,
// element k of a thread sits at position (warp*K + k)*32 + lane of the CTA's slice.  Shared by the
// tier-plan and prefetch-plan kernels.
#pragma once

#include <cuda_runtime.h>

namespace {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ int warp_incl_scan_i(int v, int lane) {
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        int t = __shfl_up_sync(kFull, v, s);
        if (lane >= s) v += t;
    }
    return v;
}

// Inclusive scan of three per-element int32 values over the CTA's T*K elements laid out as
// (warp, round, lane); returns inclusive values in place and CTA totals in tot[3].
template <int T, int K>
__device__ __forceinline__ void cta_scan3(int (&a)[K], int (&b)[K], int (&c)[K], int *tot, int (*ws)[3]) {
    constexpr int W = T / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int ra = 0, rb = 0, rc = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int ia = warp_incl_scan_i(a[k], lane), ib = warp_incl_scan_i(b[k], lane),
                  ic = warp_incl_scan_i(c[k], lane);
        a[k] = ra + ia;
        b[k] = rb + ib;
        c[k] = rc + ic;
        ra += __shfl_sync(kFull, ia, 31);
        rb += __shfl_sync(kFull, ib, 31);
        rc += __shfl_sync(kFull, ic, 31);
    }
    if (lane == 0) { ws[warp][0] = ra; ws[warp][1] = rb; ws[warp][2] = rc; }
    __syncthreads();
    if (warp == 0) {
        const bool in = lane < W;
        const int va = in ? ws[lane][0] : 0, vb = in ? ws[lane][1] : 0, vc = in ? ws[lane][2] : 0;
        const int ja = warp_incl_scan_i(va, lane), jb = warp_incl_scan_i(vb, lane), jc = warp_incl_scan_i(vc, lane);
        if (in) { ws[lane][0] = ja - va; ws[lane][1] = jb - vb; ws[lane][2] = jc - vc; }
        if (lane == 31) { ws[32][0] = ja; ws[32][1] = jb; ws[32][2] = jc; }
    }
    __syncthreads();
    const int oa = ws[warp][0], ob = ws[warp][1], oc = ws[warp][2];
#pragma unroll
    for (int k = 0; k < K; ++k) { a[k] += oa; b[k] += ob; c[k] += oc; }
    tot[0] = ws[32][0]; tot[1] = ws[32][1]; tot[2] = ws[32][2];
    __syncthreads();
}

// Sum of M int64 partials over the CTA; the totals land in every thread.
template <int T, int M>
__device__ __forceinline__ void cta_sum(long long (&v)[M], long long (*ws)[8]) {
    constexpr int W = T / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) v[m] += __shfl_xor_sync(kFull, v[m], s);
    if (lane == 0)
        for (int m = 0; m < M; ++m) ws[warp][m] = v[m];
    __syncthreads();
#pragma unroll
    for (int m = 0; m < M; ++m) {
        long long t = lane < W ? ws[lane][m] : 0;
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) t += __shfl_xor_sync(kFull, t, s);
        v[m] = t;
    }
    __syncthreads();
}


// Inclusive scan of one int64 value per element over the CTA's T*K elements; CTA total returned.
template <int T, int K>
__device__ __forceinline__ long long cta_scan_ll(long long (&a)[K], long long *ws) {
    constexpr int W = T / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    long long run = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        long long v = a[k];
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            long long t = __shfl_up_sync(kFull, v, s);
            if (lane >= s) v += t;
        }
        a[k] = run + v;
        run += __shfl_sync(kFull, v, 31);
    }
    if (lane == 0) ws[warp] = run;
    __syncthreads();
    if (warp == 0) {
        const long long t = lane < W ? ws[lane] : 0;
        long long v = t;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            long long u = __shfl_up_sync(kFull, v, s);
            if (lane >= s) v += u;
        }
        if (lane < W) ws[lane] = v - t;
        if (lane == 31) ws[32] = v;
    }
    __syncthreads();
    const long long off = ws[warp];
#pragma unroll
    for (int k = 0; k < K; ++k) a[k] += off;
    const long long total = ws[32];
    __syncthreads();
    return total;
}

}  // namespace
