// Read-only streaming probe of bench.py: the speed at which this GPU reads a buffer once with nothing else to
// do.  Not part of the HVD library and not a step of the method: the benchmark runs it over the same logits
// buffers as the verification kernel, so that the kernel's GB/s can be read against what a plain read loop
// reaches on the same part, next to the copy bandwidth and the nominal figure.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeLoads = 8;  // 128-bit loads in flight per thread

__global__ void __launch_bounds__(kProbeThreads) read_probe_kernel(const uint4* __restrict__ p, size_t n_vec,
                                                                   unsigned long long* sink) {
    const size_t stride = (size_t)gridDim.x * kProbeThreads;
    size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
    uint32_t m = 0;
    for (; i + (kProbeLoads - 1) * stride < n_vec; i += kProbeLoads * stride) {
        uint4 x[kProbeLoads];
#pragma unroll
        for (int u = 0; u < kProbeLoads; ++u)
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(x[u].x), "=r"(x[u].y), "=r"(x[u].z), "=r"(x[u].w)
                         : "l"(p + i + u * stride));
#pragma unroll
        for (int u = 0; u < kProbeLoads; ++u) m = max(max(m, max(x[u].x, x[u].y)), max(x[u].z, x[u].w));
    }
    for (; i < n_vec; i += stride) {
        const uint4 x = __ldg(p + i);
        m = max(max(m, max(x.x, x.y)), max(x.z, x.w));
    }
    m = __reduce_max_sync(0xffffffffu, m);
    if ((threadIdx.x & 31) == 0) atomicMax(sink, (unsigned long long)m);  // keeps the loads alive
}

}  // namespace

// Reads the first bytes / 16 * 16 bytes of buf (DEVICE, 16-byte aligned) once and leaves their maximum word in
// *sink (DEVICE, 8 bytes).  Enqueues one kernel on `stream` (a cudaStream_t) with `grid` CTAs; returns the CUDA
// error code of the launch (0 = success), -1 for a bad argument.
extern "C" __attribute__((visibility("default"))) int bench_read_probe(const void* buf, int64_t bytes, void* sink,
                                                                        int grid, void* stream) {
    if (!buf || !sink || bytes < 0 || grid < 1 || (reinterpret_cast<uintptr_t>(buf) & 15)) return -1;
    read_probe_kernel<<<grid, kProbeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(buf), (size_t)bytes / 16, static_cast<unsigned long long*>(sink));
    return (int)cudaGetLastError();
}
