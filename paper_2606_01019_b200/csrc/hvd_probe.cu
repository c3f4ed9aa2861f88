// Read-only streaming probe: the speed at which this GPU reads a buffer once with nothing else to do.
// Not a step of the method: the benchmark runs it over the same logits buffers as the verification
// kernel, so that the kernel's GB/s can be read against what a plain read loop reaches on the same
// part, next to the copy bandwidth and the nominal figure.
#include "hvd_internal.cuh"

namespace hvd {
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

hvd_status launch_read_probe(hvd_ctx* ctx, const void* buf, int64_t bytes, cudaStream_t stream) {
    const size_t n_vec = (size_t)bytes / 16;
    const int grid = ctx->num_sms * 8;
    read_probe_kernel<<<grid, kProbeThreads, 0, stream>>>(static_cast<const uint4*>(buf), n_vec, ctx->probe_sink);
    HVD_CUDA_TRY(ctx, cudaGetLastError());
    return HVD_OK;
}

}  // namespace hvd
