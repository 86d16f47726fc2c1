// Measurement aid, not part of the method: a read-only streaming kernel that gives the HBM read ceiling of the
// GPU the benchmark runs on, in the same process and under the same clocks as the attend kernel it is compared with.
#include "common.cuh"

namespace lookat {

namespace {

constexpr int kProbeThreads = 256, kProbeUnroll = 8;

// every thread keeps kProbeUnroll independent 16-byte loads in flight; nothing is written unless the data XORs to
// a value it cannot have, which keeps the loads alive without a store stream
__global__ void __launch_bounds__(kProbeThreads) read_probe_kernel(const uint4 *__restrict__ p, size_t n16, unsigned *sink)
{
    const size_t stride = (size_t)gridDim.x * kProbeThreads;
    size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
    unsigned acc = 0;
    for (; i + (kProbeUnroll - 1) * stride < n16; i += kProbeUnroll * stride) {
        uint4 v[kProbeUnroll];
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) v[u] = __ldcs(p + i + u * stride);
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    for (; i < n16; i += stride) {
        const uint4 v = __ldcs(p + i);
        acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
    if (acc == 0x9e3779b9u && sink) *sink = acc;
}

}  // namespace

lookat_status probe_read_bandwidth(Ctx *ctx, const void *buf, size_t bytes, int reps, double *gb_per_s)
{
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return check_launch(ctx, "probe: events");
    const size_t n16 = bytes / 16;
    const int grid = ctx->sm_count * 8;
    read_probe_kernel<<<grid, kProbeThreads, 0, ctx->stream>>>(reinterpret_cast<const uint4 *>(buf), n16, nullptr);   // warm-up
    cudaEventRecord(e0, ctx->stream);
    for (int r = 0; r < reps; ++r)
        read_probe_kernel<<<grid, kProbeThreads, 0, ctx->stream>>>(reinterpret_cast<const uint4 *>(buf), n16, nullptr);
    cudaEventRecord(e1, ctx->stream);
    lookat_status st = check_launch(ctx, "read_probe_kernel");
    float ms = 0.f;
    if (st == LOOKAT_OK && (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess))
        st = check_launch(ctx, "probe: timing");
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (st != LOOKAT_OK) return st;
    ctx->launches += (uint64_t)reps;                       // check_launch counted one
    *gb_per_s = (double)n16 * 16.0 * reps / ((double)ms * 1e-3) / 1e9;
    return LOOKAT_OK;
}

}  // namespace lookat
