// BN + ReLU forward for callers that must not allocate device memory.
//
// resist_bn_relu_forward() obtains its reduction scratch with cudaMalloc on every call.  Some callers cannot do
// that: code that runs inside a memory pool it may not grow, a real-time loop in which an allocation (and the
// device-wide synchronisation cudaFree implies) is a latency spike, or a host framework that has handed all
// device memory to its own allocator.  This file gives them the same operation with the scratch in a fixed
// array that is part of the library image: every GPU that loads the library holds RESIST_NOALLOC_SCRATCH_BYTES
// of it until the process exits.
#include <string>
#include "runtime.h"

using namespace resist;

#define RESIST_NOALLOC_SCRATCH_BYTES (4u << 20)
constexpr size_t NOALLOC_DESC_BYTES = 256;        // the problem descriptor lives in front of the partial sums

// File-scope device array.  In HOST code this name is only a handle: the device address has to be asked for
// with cudaGetSymbolAddress (below).  Device code may name it directly (store_descriptor does).
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_DESC_BYTES + RESIST_NOALLOC_SCRATCH_BYTES];

static thread_local std::string g_noalloc_error;
extern "C" const char* resist_noalloc_last_error(void) { return g_noalloc_error.c_str(); }

// The grouped BN kernels read their problem from device memory; this writes it there without a copy call.
__global__ void store_descriptor(BnProb p) { *reinterpret_cast<BnProb*>(g_noalloc_scratch) = p; }

// One device address per GPU, looked up the first time a call runs with that GPU current.
static unsigned char* scratch_of_current_device(int* rc) {
    static unsigned char* table[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { g_noalloc_error = "cannot identify the current device"; *rc = RESIST_ECUDA; return nullptr; }
    if (!table[dev]) {
        unsigned char* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || !ptr) { g_noalloc_error = std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e); *rc = RESIST_ECUDA; return nullptr; }
        table[dev] = ptr;
    }
    *rc = RESIST_OK;
    return table[dev];
}

extern "C" int resist_bn_relu_forward_noalloc(int32_t dtype, const void* x, const float* gamma, const float* beta, void* a,
                                              float* stat, float* run_mean, float* run_var, int64_t m, int32_t C, float eps,
                                              float momentum, resist_stream stream) {
    if (!x || !gamma || !beta || !a || !stat || m < 1 || C < 1) { g_noalloc_error = "bad argument"; return RESIST_EINVAL; }
    if (dtype != RESIST_F32 && dtype != RESIST_BF16) { g_noalloc_error = "bad dtype"; return RESIST_EINVAL; }
    static_assert(sizeof(BnProb) <= NOALLOC_DESC_BYTES, "descriptor slot too small");
    cudaStream_t st = (cudaStream_t)stream;
    BnProb p{}; p.x = x; p.a = a; p.gamma = gamma; p.beta = beta; p.run_mean = run_mean; p.run_var = run_var; p.stat = stat;
    p.eps = eps; p.momentum = momentum; p.m = m; p.C = C;
    // the same chunking as resist_bn_relu_forward, so that both give the same bits
    bn_chunking(p, dtype == RESIST_BF16);
    const size_t need = (size_t)p.chunks * 2 * (size_t)C * sizeof(double);
    if (need > RESIST_NOALLOC_SCRATCH_BYTES) {
        g_noalloc_error = "needs " + std::to_string(need) + " bytes of reduction scratch (chunks x 2 x C doubles) but the built-in array holds " +
                          std::to_string((size_t)RESIST_NOALLOC_SCRATCH_BYTES) + "; use resist_bn_relu_forward";
        return RESIST_EUNSUPPORTED;
    }
    int rc = RESIST_OK;
    unsigned char* base = scratch_of_current_device(&rc);
    if (!base) return rc;
    p.partial = reinterpret_cast<double*>(base + NOALLOC_DESC_BYTES);
    // Nothing in the array has to start at zero: every partial sum the finalise step reads is written first by
    // the reduction of this same call, and the descriptor is rewritten here.
    store_descriptor<<<1, 1, 0, st>>>(p);
    const BnProb* d = reinterpret_cast<const BnProb*>(base);
    launch_bn_stats(d, 1, p.chunks, C, dtype == RESIST_BF16, st);
    launch_bn_apply(d, 1, m * C, dtype == RESIST_BF16, st);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { g_noalloc_error = std::string("launch failed: ") + cudaGetErrorString(e); return RESIST_ECUDA; }
    return RESIST_OK;
}
