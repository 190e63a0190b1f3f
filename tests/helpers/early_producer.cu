// Test helper, not part of the library: a producer kernel of the kind some GEMM and normalisation
// kernels are -- it tells the stream that dependents may start ("griddepcontrol.launch_dependents")
// long before its last store.  It idles for `delay_cycles` (a fixed delay on the SM clock, not a wait on
// anything) and only then copies `src` over `dst`.  A consumer that is launched with programmatic
// stream serialization and reads `dst` without waiting for this kernel's completion sees the old bytes.
#include <cuda_runtime.h>
#include <stdint.h>

__global__ void early_producer_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, long long n_units,
                                      long long delay_cycles)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long t0 = clock64();
    while (clock64() - t0 < delay_cycles) { }
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_units; i += stride)
        dst[i] = src[i];
}

// bytes: a multiple of 16; both pointers 16-byte aligned.  Returns the CUDA error code of the launch.
extern "C" int launch_early_producer(const void *src, void *dst, long long bytes, long long delay_cycles, void *stream)
{
    early_producer_kernel<<<32, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4 *>(src), static_cast<uint4 *>(dst), bytes / 16, delay_cycles);
    return static_cast<int>(cudaGetLastError());
}
