// Test-only kernels (not part of the library): a producer that releases its programmatic dependents before it
// writes, and a launch that makes the library's bounded barrier wait run out.  Built by tests/cuda_helpers.py.
#include <cuda_runtime.h>
#include <stdint.h>

#include "grid_barrier.cuh"

namespace {

// Releases the kernels queued behind it at once, idles for `delay` cycles of the SM clock (bounded by the host
// wrapper), and only then copies src to dst: whatever reads dst before this grid has finished sees stale data.
__global__ void early_trigger_copy_kernel(const float* src, float* dst, int64_t n, long long delay) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const long long t0 = clock64();
    while (clock64() - t0 < delay) { }
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) dst[i] = src[i];
}

// Every CTA arrives once at a barrier that expects one member more than the grid has: nobody completes it, every
// wait runs out after `polls` polls, sets the workspace's error flag and returns.  returned[cta] = 1 + what the
// barrier reported (so 1 = "gave up", and 0 would mean the CTA never came back).
__global__ void barrier_timeout_kernel(profk::WsHeader* header, uint32_t members, uint32_t polls, uint32_t* returned) {
    const bool ok = profk::cta_group_barrier(&header->bar_count, &header->error, members, polls);
    if (threadIdx.x == 0) returned[blockIdx.x] = 1u + (ok ? 1u : 0u);
}

}  // namespace

extern "C" int profk_test_early_trigger_copy_f32(const float* src, float* dst, int64_t n, int64_t delay_cycles, void* stream) {
    if (!src || !dst || n < 1 || delay_cycles < 0 || delay_cycles > (1 << 22)) return -1;      // at most ~2 ms of idling
    early_trigger_copy_kernel<<<592, 256, 0, static_cast<cudaStream_t>(stream)>>>(src, dst, n, (long long)delay_cycles);
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

// `workspace` is the device allocation registered with profk_set_workspace (its header comes first); `returned`
// holds `ctas` words.  ctas <= 64 keeps all CTAs co-resident; members must exceed ctas; polls <= 2^16.
extern "C" int profk_test_barrier_timeout(void* workspace, uint32_t ctas, uint32_t members, uint32_t polls, uint32_t* returned, void* stream) {
    if (!workspace || !returned || ctas < 1 || ctas > 64 || members <= ctas || polls > (1u << 16)) return -1;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, sizeof(profk::WsHeader), st) != cudaSuccess) return -3;
    if (cudaMemsetAsync(returned, 0, ctas * sizeof(uint32_t), st) != cudaSuccess) return -3;
    barrier_timeout_kernel<<<ctas, 128, 0, st>>>(static_cast<profk::WsHeader*>(workspace), members, polls, returned);
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}
