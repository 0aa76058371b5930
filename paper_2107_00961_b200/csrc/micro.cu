// Micro-benchmark of the tcgen05.mma issue and execution rate on one SM, as a function of the MMA's N, of the operand layout in
// shared memory and of the number of issuing threads.  It backs the tile-shape choices of the convolution kernels with numbers
// measured on the device at hand: one CTA per SM allocates tensor memory, leaves its shared memory as it finds it (the values do
// not matter for the rate, and every address the descriptors name lies inside the CTA's own allocation), issues `reps` MMAs of
// shape 128 x N x 16 (bf16 -> fp32) back to back, commits them to an mbarrier and waits (bounded) for their completion; the time
// between the first issue and the completion is taken with the SM's clock.
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/resist.h"

namespace resist_micro {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo, uint32_t swizzle) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) | ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46) |
           ((uint64_t)swizzle << 61);
}

struct Args { int n, layout, reps, issuers, alternate; long long* cycles; int* status; };
// layout 0: K-major, no swizzle (8 x 16-byte core matrices, planes of 8 channels); 1: K-major, 128-byte swizzle (rows of 64 channels,
// the four K = 16 steps of a row walked in turn); 2: as 1 but every MMA reads the same 32-byte step; 3: MN-major, 128-byte swizzle.
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(const Args a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bar[2];
    __shared__ uint32_t tmem_s;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&bar[i])), "r"(1) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_s)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_s;
    // operands: A = 128 rows, B = n rows (or the MN-major equivalents), both inside 64 KB from `base`
    const uint32_t a_addr = base, b_addr = base + 32768;
    const int n = a.n;
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (a.layout == 3 ? (1u << 15) | (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
    long long t0 = 0, t1 = 0;
    if (warp < a.issuers && lane == 0) {
        const int me = warp;
        t0 = clock64();
        for (int r = me; r < a.reps; r += a.issuers) {
            const uint32_t step = (uint32_t)(r & 3);
            uint64_t ad, bd;
            if (a.layout == 0) { ad = make_desc(a_addr + step * 4096u, 2048, 128, 0); bd = make_desc(b_addr + step * 8192u, 4096, 128, 0); }        // planes: LBO = next 8 channels, SBO = next 8 rows
            else if (a.layout == 1) { ad = make_desc(a_addr + step * 32u, 16, 1024, 2); bd = make_desc(b_addr + step * 32u, 16, 1024, 2); }
            else if (a.layout == 2) { ad = make_desc(a_addr, 16, 1024, 2); bd = make_desc(b_addr, 16, 1024, 2); }
            else { ad = make_desc(a_addr + step * 2048u, 16384, 1024, 2); bd = make_desc(b_addr + step * 2048u, 8192, 1024, 2); }     // MN-major: 16 rows per step, 64-column blocks
            const uint32_t d = tmem + (a.alternate ? (uint32_t)(r & 1) * 256u : 0u);
            const uint32_t acc = r >= 2 ? 1u : 0u;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                         ::"r"(d), "l"(ad), "l"(bd), "r"(idesc), "r"(acc) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bar[me])) : "memory");
        bool done = false;
        for (uint32_t i = 0; i < (1u << 22) && !done; ++i) {
            uint32_t ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(smem_u32(&bar[me])), "r"(0) : "memory");
            done = ok != 0;
        }
        t1 = clock64();
        if (!done) atomicExch(a.status, 1);
        if (blockIdx.x == 0) a.cycles[me] = t1 - t0;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

}  // namespace resist_micro

// n: MMA N (16..256, multiple of 16); layout 0..3 (see the kernel); reps: MMAs issued per CTA; issuers: 1 or 2 issuing threads (warps);
// alternate: 1 = consecutive MMAs go to two different accumulators.  *cycles_per_mma (host) receives SM clocks per MMA of CTA 0,
// first issue to completion.  Allocates a few bytes with cudaMalloc and synchronises the device.
extern "C" int resist_micro_mma_rate(int32_t n, int32_t layout, int32_t reps, int32_t issuers, int32_t alternate, double* cycles_per_mma) {
    using namespace resist_micro;
    if (n < 16 || n > 256 || n % 16 || layout < 0 || layout > 3 || reps < 4 || issuers < 1 || issuers > 2 || !cycles_per_mma) return RESIST_EINVAL;
    char* blob = nullptr;
    if (cudaMalloc(&blob, 256) != cudaSuccess) return RESIST_ENOMEM;
    cudaMemset(blob, 0, 256);
    Args a{n, layout, reps, issuers, alternate, (long long*)blob, (int*)(blob + 64)};
    static bool configured = false;
    if (!configured) { cudaFuncSetAttribute(mma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024); configured = true; }
    int dev = 0, sms = 1; cudaGetDevice(&dev); cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    mma_rate_kernel<<<sms, 128, 120 * 1024, 0>>>(a);
    long long cyc[2] = {0, 0}; int st = 0;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(cyc, blob, 16, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(&st, blob + 64, 4, cudaMemcpyDeviceToHost);
    cudaFree(blob);
    if (e != cudaSuccess) return RESIST_ECUDA;
    if (st) return RESIST_ETIMEOUT;
    *cycles_per_mma = (double)(cyc[0] > cyc[1] ? cyc[0] : cyc[1]) / (double)reps;
    return RESIST_OK;
}
