// Test-only helper (not part of the library): a finite kernel that occupies SMs and their shared
// memory for a bounded number of clocks, so that a test can run the copy kernels on a busy GPU.
// It spins on the clock only, never on memory that somebody else writes, and always ends by itself.
#include <cuda_runtime.h>

__global__ void occupy_kernel(long long clocks) {
    extern __shared__ unsigned char hold[];
    const long long t0 = clock64();
    while (clock64() - t0 < clocks) __nanosleep(2000);
    if (clocks < 0) hold[0] = 0;   // never taken; keeps the shared array referenced
}

// Launches `ctas` CTAs of 64 threads holding `smem_bytes` of shared memory each for about `clocks`
// SM clocks on `stream`.  Returns the cudaError_t of the launch.
extern "C" int filler_launch(int ctas, int smem_bytes, long long clocks, void *stream) {
    if (clocks > 400000000LL) clocks = 400000000LL;   // a fifth of a second at most
    cudaError_t e = cudaFuncSetAttribute(occupy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return (int)e;
    occupy_kernel<<<ctas, 64, smem_bytes, (cudaStream_t)stream>>>(clocks);
    return (int)cudaGetLastError();
}
