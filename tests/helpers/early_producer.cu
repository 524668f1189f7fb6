// Test helper, not part of the library: a producer kernel that behaves like a GEMM epilogue
// written for programmatic dependent launch. It releases the kernels behind it in the stream
// FIRST, idles for a bounded number of clock cycles, and only then writes its output. A
// consumer that reads that output before its own griddepcontrol.wait sees what was there before.
#include <cuda_runtime.h>
#include <stdint.h>

extern "C" __global__ void early_producer_kernel(uint4 *dst, const uint4 *src, size_t n, long long delay)
{
    asm volatile("griddepcontrol.launch_dependents;");
    const long long t0 = clock64();
    while (clock64() - t0 < delay) { }                      // a fixed number of cycles: nothing is waited for
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}

// dst, src: device pointers, 16-byte aligned; bytes: a multiple of 16. Returns the CUDA error code.
extern "C" int early_producer(void *dst, const void *src, size_t bytes, long long delay_cycles, void *stream)
{
    if (bytes % 16 != 0 || ((uintptr_t)dst & 15) || ((uintptr_t)src & 15)) return -1;
    // A multiprocessor keeps the split between L1 and shared memory of the kernel that runs on it:
    // blocks of a kernel that needs shared memory cannot join one that was set up with none. Ask
    // for the largest shared-memory share, so that any consumer's blocks can become resident
    // beside this kernel's (which is the situation the test is about).
    cudaError_t e = cudaFuncSetAttribute(early_producer_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return (int)e;
    early_producer_kernel<<<148, 256, 0, (cudaStream_t)stream>>>((uint4 *)dst, (const uint4 *)src, bytes / 16, delay_cycles);
    return (int)cudaGetLastError();
}
