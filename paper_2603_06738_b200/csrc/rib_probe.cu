// Two small measurement / self-test kernels of the library (not part of the method):
//   rib_exp_probe        how many exponentials per second the exp (MUFU) pipe of this GPU delivers, which
//                        bounds the forward pass at 32-channel heads (one exponential per 160 tensor flops);
//   rib_wait_probe       one CTA that waits, with a short limit, for an mbarrier nobody arrives at, so that the
//                        path every bounded wait of the tcgen05 kernels takes when it gives up (abort flag,
//                        status word, common tail that frees tensor memory) can be exercised without a fault.
#include "rib_common.cuh"
#include "sm100_primitives.cuh"

namespace rib {
namespace {

using namespace sm100;

constexpr int kProbeThreads = 512;
constexpr int kProbeUnroll = 8;      // independent exponentials in flight per thread

// iters * kProbeUnroll exponentials per thread on register values that change every round
__global__ void __launch_bounds__(kProbeThreads) rib_exp_probe_kernel(float* sink, int iters)
{
    float x[kProbeUnroll];
#pragma unroll
    for (int k = 0; k < kProbeUnroll; ++k) x[k] = -0.001f * (float)(threadIdx.x + 32 * k + 1);
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int k = 0; k < kProbeUnroll; ++k) x[k] = ex2_approx(x[k]) - 1.25f;     // stays in (-1.25, -0.25]
    }
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < kProbeUnroll; ++k) s += x[k];
    if (s == 12345.678f) sink[0] = s;        // keeps the loop alive; never true
}

// The give-up path of the tcgen05 kernels in miniature: allocate tensor memory, wait (bounded by limit_ns) for a
// phase that never completes, leave through a tail that frees the tensor memory.
__global__ void __launch_bounds__(128) rib_wait_probe_kernel(int* status, unsigned long long limit_ns)
{
    __shared__ uint64_t bar_mem;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar_mem), 1);
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 32);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    // every warp waits; the first one whose limit runs out raises the abort flag and the others follow it
    mbar_wait_limited(smem_u32(&bar_mem), 0, &abort_flag, status, limit_ns);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, 32);
    }
}

}  // namespace

cudaError_t exp_probe(float* sink, int blocks, int iters, cudaStream_t stream)
{
    rib_exp_probe_kernel<<<blocks, kProbeThreads, 0, stream>>>(sink, iters);
    return cudaGetLastError();
}

long long exp_probe_count(int blocks, int iters) { return (long long)blocks * kProbeThreads * kProbeUnroll * iters; }

cudaError_t wait_probe(int* status, unsigned long long limit_ns, cudaStream_t stream)
{
    rib_wait_probe_kernel<<<1, 128, 0, stream>>>(status, limit_ns);
    return cudaGetLastError();
}

}  // namespace rib
