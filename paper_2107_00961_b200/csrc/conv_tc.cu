// Tensor-core convolutions for sm_100a: implicit GEMM on tcgen05.mma with the accumulator in TMEM and the
// operands staged in shared memory by TMA.
//
// Forward and dgrad of a stride-1 k x k convolution (k = 1 or 3) share one kernel.  The output tile is 128
// consecutive positions of one image in "padded-flat" order (row-major over rows of W + 2*pad positions; the
// 2*pad extra positions per row are computed and thrown away).  In that order the operand of filter tap (r,s) is
// the SAME pixel run shifted by r*(W+2*pad)+s positions, so the input halo is fetched ONCE per tile (TMA box
// with out-of-bounds zero fill = the zero padding) and all k*k taps read it through shifted shared-memory
// descriptors.  Shared memory holds the pixels as planes of 8 channels (16 bytes per pixel per plane), which is
// the canonical no-swizzle K-major layout of the MMA: 8 pixels x 16 B form one core matrix, any 16-byte pixel
// offset is a legal start address.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..5 = epilogue
// (TMEM -> registers -> scale, residual add, bf16 -> global).  Every wait is bounded: on expiry the kernel
// records the place in the status word, drains, frees its TMEM and returns.
#include <cuda.h>
#include <cstdio>
#include <cstring>
#include "internal.h"

namespace resist {

// ------------------------------------------------------------------------------------------------ device helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait: false when the barrier did not flip within the limit
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i > 64) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    // no-swizzle matrix descriptor: start >> 4 | LBO >> 4 at bit 16 | SBO >> 4 at bit 32 | version 1 at bit 46
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                   "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr));
}

// One tensor-core convolution problem.  The two tensor maps come first so that each is 64-byte aligned.
struct alignas(64) TcProb {
    CUtensorMap map_a;        // activations (forward: a; dgrad: dy) viewed as (channel, x, y, image)
    CUtensorMap map_b;        // weights viewed as (8 input channels, output channel, input-channel group, tap)
    const __nv_bfloat16* add; __nv_bfloat16* out;
    int* status;
    int H, W, Wp, pad, taps, flip;          // image extent (1x1 layers: one long row), padded width, taps = k*k
    int n_img, tiles_per_img, tiles_n;
    int ncol;                               // channels of the output tensor
    int n_tile;                             // MMA N: output channels per CTA (multiple of 16, <= 256)
    int kc, nchunks;                        // reduction channels per pipeline stage, number of stages' worth
    int box_w, box_h;                       // activation box (pixels)
    int plane_bytes;                        // one 8-channel plane of the activation box, padded
    int a_stage_bytes, b_stage_bytes, b_tap_bytes;
    int b_mn_major;                         // 0: forward (weights K-major); 1: dgrad (weights MN-major)
    int tmem_cols; int flat;                // flat = 1: 1x1 layer, tile = 128 consecutive pixels of the whole tensor
    int stages;                             // pipeline depth: 1 when the reduction fits one stage, else 2
    int os, P, Q;                           // output stride: only positions (i,j) with i,j multiples of os are stored, as pixel (i/os, j/os) of a P x Q image
    float scale;
};

constexpr int TC_THREADS = 192;
constexpr int TC_STAGES = 2;

__global__ void __launch_bounds__(TC_THREADS) conv_tc_kernel(const TcProb* __restrict__ probs) {
    const TcProb& p = probs[blockIdx.y];
    const int tiles = p.n_img * p.tiles_per_img * p.tiles_n;
    if ((int)blockIdx.x >= tiles) return;
    const int tn = blockIdx.x % p.tiles_n;
    const int tm = blockIdx.x / p.tiles_n;
    const int img = tm / p.tiles_per_img, t_in = tm % p.tiles_per_img;
    const int pos0 = t_in * 128;                                  // first padded-flat position of this tile
    const int row0 = p.flat ? 0 : pos0 / p.Wp;                    // first output row touched
    const int a_off = p.flat ? 0 : pos0 - row0 * p.Wp;            // tile start inside the box, tap (0,0)

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    __shared__ __align__(8) uint64_t bars[2 * TC_STAGES + 1];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[TC_STAGES]), bar_acc = smem_u32(&bars[2 * TC_STAGES]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_s;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            for (int c = 0; c < p.nchunks; ++c) {
                const int s = c % p.stages, it = c / p.stages;
                if (it > 0 && !mbar_wait(bar_empty + 8 * s, (it - 1) & 1)) { atomicExch(&abort_s, 1); atomicExch(p.status, 1); break; }
                const uint32_t a_dst = smem_u32(smem + s * stage_bytes), b_dst = a_dst + p.a_stage_bytes;
                mbar_expect_tx(bar_full + 8 * s, (uint32_t)((p.kc / 8) * p.box_w * p.box_h * 16 + p.taps * p.b_tap_bytes));
                const int x0 = p.flat ? pos0 : -p.pad, y0 = p.flat ? 0 : row0 - p.pad;
                for (int pl = 0; pl < p.kc / 8; ++pl)
                    tma_load_4d(a_dst + pl * p.plane_bytes, &p.map_a, bar_full + 8 * s, c * p.kc + pl * 8, x0, y0, img);
                if (!p.b_mn_major) tma_load_4d(b_dst, &p.map_b, bar_full + 8 * s, 0, tn * p.n_tile, c * (p.kc / 8), 0);
                else tma_load_4d(b_dst, &p.map_b, bar_full + 8 * s, 0, c * p.kc, tn * (p.n_tile / 8), 0);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            // instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B K-major or MN-major, N, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.b_mn_major << 16) |
                                   ((uint32_t)(p.n_tile >> 3) << 17) | ((128u >> 4) << 24);
            const int ksz = p.taps == 9 ? 3 : 1;
            bool ok = true;
            for (int c = 0; c < p.nchunks && ok; ++c) {
                const int s = c % p.stages, it = c / p.stages;
                if (!mbar_wait(bar_full + 8 * s, it & 1)) { atomicExch(&abort_s, 1); atomicExch(p.status, 2); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_base = smem_u32(smem + s * stage_bytes), b_base = a_base + p.a_stage_bytes;
                for (int t = 0; t < p.taps; ++t) {
                    const int r = t / ksz, q = t % ksz;
                    const int shift = p.flip ? ((ksz - 1 - r) * p.Wp + (ksz - 1 - q)) : (r * p.Wp + q);
                    for (int k16 = 0; k16 < p.kc / 16; ++k16) {
                        const uint64_t ad = smem_desc(a_base + 2 * k16 * p.plane_bytes + (a_off + shift) * 16, p.plane_bytes, 128);
                        uint64_t bd;
                        if (!p.b_mn_major) bd = smem_desc(b_base + t * p.b_tap_bytes + 2 * k16 * p.n_tile * 16, p.n_tile * 16, 128);
                        else bd = smem_desc(b_base + t * p.b_tap_bytes + k16 * 256, 128, p.kc * 16);
                        umma_bf16(tmem_d, ad, bd, idesc, (c | t | k16) ? 1u : 0u);
                    }
                }
                umma_commit(bar_empty + 8 * s);          // stage reusable once these MMAs have read it
            }
            if (ok) umma_commit(bar_acc);                // accumulator complete
        }
    } else {
        // ---------------------------------------------------------------- epilogue: 4 warps, one TMEM lane quadrant each
        const int quad = warp & 3;
        const int m = quad * 32 + lane;                  // row of the tile = TMEM lane
        bool ok = mbar_wait(bar_acc, 0);
        ok = __all_sync(0xffffffffu, ok);                // tcgen05.ld below is warp-collective
        if (!ok) { atomicExch(&abort_s, 1); atomicExch(p.status, 3); }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // padded-flat position -> output pixel
        long long pix = -1;
        if (p.flat) { const long long g = (long long)pos0 + m; if (g < (long long)p.W) pix = g; }
        else {
            const int pos = pos0 + m, i = pos / p.Wp, j = pos - i * p.Wp;
            if (i < p.H && j < p.W) {
                if (p.os == 1) pix = ((long long)img * p.H + i) * p.W + j;
                else if (i % p.os == 0 && j % p.os == 0) pix = ((long long)img * p.P + i / p.os) * p.Q + j / p.os;   // strided layer
            }
        }
        if (ok) {
            for (int c0 = 0; c0 < p.n_tile; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (pix >= 0) {
                    const long long o = pix * p.ncol + tn * p.n_tile + c0;
                    float f[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) f[k] = __uint_as_float(v[k]) * p.scale;
                    if (p.add) {
                        const uint4 a0 = *reinterpret_cast<const uint4*>(p.add + o), a1 = *reinterpret_cast<const uint4*>(p.add + o + 8);
                        const uint32_t aw[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            f[2 * k] += __uint_as_float(aw[k] << 16);
                            f[2 * k + 1] += __uint_as_float(aw[k] & 0xFFFF0000u);
                        }
                    }
                    uint32_t w[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
                        w[k] = *reinterpret_cast<uint32_t*>(&h);
                    }
                    *reinterpret_cast<uint4*>(p.out + o) = make_uint4(w[0], w[1], w[2], w[3]);
                    *reinterpret_cast<uint4*>(p.out + o + 8) = make_uint4(w[4], w[5], w[6], w[7]);
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(p.tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------ zero stuffing
// Backward of a stride-2 layer runs as a stride-1 problem on dy spread out to the input resolution:
// up[n, 2p, 2q, :] = dy[n, p, q, :], zero elsewhere.  Then dgrad(up) and wgrad(a, up) at stride 1 are the
// stride-2 dgrad and wgrad, term for term.
__global__ void __launch_bounds__(256) zero_stuff_kernel(const UpProb* __restrict__ probs) {
    const UpProb& p = probs[blockIdx.y];
    const int G = p.K >> 3;
    const long long nv = (long long)p.N * p.H * p.W * G;
    const uint4* src = reinterpret_cast<const uint4*>(p.src);
    uint4* dst = reinterpret_cast<uint4*>(p.dst);
    for (long long v = blockIdx.x * (long long)blockDim.x + threadIdx.x; v < nv; v += (long long)gridDim.x * blockDim.x) {
        const int g = (int)(v % G); long long t = v / G; const int w = (int)(t % p.W); t /= p.W; const int h = (int)(t % p.H); const int n = (int)(t / p.H);
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (!(h & 1) && !(w & 1) && (h >> 1) < p.P && (w >> 1) < p.Q) val = src[(((long long)n * p.P + (h >> 1)) * p.Q + (w >> 1)) * G + g];
        dst[v] = val;
    }
}
void launch_zero_stuff(const UpProb* d, int nprob, long long max_vecs, cudaStream_t s) {
    long long gx = (max_vecs + 255) / 256; if (gx > 148 * 16) gx = 148 * 16; if (gx < 1) gx = 1;
    zero_stuff_kernel<<<dim3((unsigned)gx, nprob), 256, 0, s>>>(d);
}

// ------------------------------------------------------------------------------------------------ wgrad
// dw[k][r][s][c] = sum over output pixels of dy[pix][k] * a[pix + shift(r,s)][c].  The reduction runs over the
// padded-flat pixel positions of the forward kernel, 128 per pipeline stage: D[cout (128 lanes), cin] per tap,
// A = dy^T and B = shifted a, both MN-major straight from their 8-channel planes.  dy is fetched with a box that
// starts at column 0, so the pad positions of every row and the rows past the image read as zero and add nothing.
// A CTA accumulates a range of pixel tiles for a group of taps and writes an fp32 partial; a second kernel adds
// the partials in a fixed order.
struct alignas(64) TcWgradProb {
    CUtensorMap map_dy;       // (channel k, x, y, image)
    CUtensorMap map_a;        // (channel c, x, y, image)
    float* partial;           // [splits][taps][cout][cin]
    float* out;               // [cout][taps][cin]
    int* status;
    int H, W, Wp, pad, taps, ksz, flat;
    int n_img, tiles_per_img, pixel_tiles;       // pixel tiles in total = n_img * tiles_per_img
    int cout, cin, m_tiles, n_tile, n_tiles;     // cout tiles of 128 rows, cin tiles of n_tile columns
    int tap_groups, taps_per_group, splits, tiles_per_split;
    int box_w, box_h_a, box_h_dy;
    int plane_a, plane_dy;                       // bytes of one 8-channel plane
    int dy_planes, a_planes;                     // planes fetched per stage
    int stage_bytes, stages, tmem_cols;
};

__global__ void __launch_bounds__(TC_THREADS) conv_wgrad_tc_kernel(const TcWgradProb* __restrict__ probs) {
    const TcWgradProb& p = probs[blockIdx.y];
    const int ctas = p.m_tiles * p.n_tiles * p.tap_groups * p.splits;
    if ((int)blockIdx.x >= ctas) return;
    int id = blockIdx.x;
    const int split = id % p.splits; id /= p.splits;
    const int tg = id % p.tap_groups; id /= p.tap_groups;
    const int tn = id % p.n_tiles; const int tm = id / p.n_tiles;
    const int t_begin = split * p.tiles_per_split;
    int t_end = t_begin + p.tiles_per_split; if (t_end > p.pixel_tiles) t_end = p.pixel_tiles;
    const int tap0 = tg * p.taps_per_group;
    int ntap = p.taps - tap0; if (ntap > p.taps_per_group) ntap = p.taps_per_group;
    const int nt = t_end - t_begin;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    __shared__ __align__(8) uint64_t bars[2 * 4 + 1];
    __shared__ uint32_t tmem_base_s;
    const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[4]), bar_acc = smem_u32(&bars[8]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_s;

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < nt; ++i) {
                const int s = i % p.stages, it = i / p.stages;
                if (it > 0 && !mbar_wait(bar_empty + 8 * s, (it - 1) & 1)) { atomicExch(p.status, 11); break; }
                const int t = t_begin + i, img = t / p.tiles_per_img, pos0 = (t % p.tiles_per_img) * 128;
                const int row0 = p.flat ? 0 : pos0 / p.Wp;
                const uint32_t dy_dst = smem_u32(smem + s * p.stage_bytes), a_dst = dy_dst + p.dy_planes * p.plane_dy;
                mbar_expect_tx(bar_full + 8 * s, (uint32_t)(p.dy_planes * p.box_w * p.box_h_dy * 16 + p.a_planes * p.box_w * p.box_h_a * 16));
                for (int pl = 0; pl < p.dy_planes; ++pl)
                    tma_load_4d(dy_dst + pl * p.plane_dy, &p.map_dy, bar_full + 8 * s, tm * 128 + pl * 8, p.flat ? pos0 : 0, row0, img);
                for (int pl = 0; pl < p.a_planes; ++pl)
                    tma_load_4d(a_dst + pl * p.plane_a, &p.map_a, bar_full + 8 * s, tn * p.n_tile + pl * 8, p.flat ? pos0 : -p.pad,
                                p.flat ? 0 : row0 - p.pad, img);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // fp32 accumulate, bf16 x bf16, A and B MN-major, N = n_tile, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(p.n_tile >> 3) << 17) | ((128u >> 4) << 24);
            bool ok = true;
            for (int i = 0; i < nt && ok; ++i) {
                const int s = i % p.stages, it = i / p.stages;
                if (!mbar_wait(bar_full + 8 * s, it & 1)) { atomicExch(p.status, 12); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int pos0 = ((t_begin + i) % p.tiles_per_img) * 128;
                const int off = p.flat ? 0 : pos0 % p.Wp;
                const uint32_t dy_base = smem_u32(smem + s * p.stage_bytes), a_base = dy_base + p.dy_planes * p.plane_dy;
                for (int tt = 0; tt < ntap; ++tt) {
                    const int t = tap0 + tt, r = t / p.ksz, q = t % p.ksz;
                    for (int k16 = 0; k16 < 8; ++k16) {
                        const uint64_t ad = smem_desc(dy_base + (off + k16 * 16) * 16, 128, p.plane_dy);
                        const uint64_t bd = smem_desc(a_base + (off + r * p.Wp + q + k16 * 16) * 16, 128, p.plane_a);
                        umma_bf16(tmem_d + (uint32_t)(tt * p.n_tile), ad, bd, idesc, (i | k16) ? 1u : 0u);
                    }
                }
                umma_commit(bar_empty + 8 * s);
            }
            if (ok) umma_commit(bar_acc);
        }
    } else {
        const int quad = warp & 3, m = quad * 32 + lane;
        bool ok = nt > 0 ? mbar_wait(bar_acc, 0) : true;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) atomicExch(p.status, 13);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int k = tm * 128 + m;
        if (ok && quad * 32 < p.cout - tm * 128) {            // warp-uniform: this lane quadrant holds real output channels
            for (int tt = 0; tt < ntap; ++tt) {
                float* dst = p.partial + (((long long)split * p.taps + tap0 + tt) * p.cout + k) * p.cin + tn * p.n_tile;
                for (int c0 = 0; c0 < p.n_tile; c0 += 16) {
                    uint32_t v[16];
                    if (nt > 0) { tmem_ld16(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(tt * p.n_tile + c0), v);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
                    else { for (int j = 0; j < 16; ++j) v[j] = 0u; }
                    if (k < p.cout) {
#pragma unroll
                        for (int j = 0; j < 16; j += 4)
                            *reinterpret_cast<uint4*>(dst + c0 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(p.tmem_cols) : "memory");
    }
}

// out[k][t][c] = sum over splits (ascending) of partial[split][t][k][c]
__global__ void __launch_bounds__(256) wgrad_tc_reduce_kernel(const TcWgradProb* __restrict__ probs) {
    const TcWgradProb& p = probs[blockIdx.y];
    const long long n = (long long)p.taps * p.cout * p.cin;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % p.cin); const long long r = i / p.cin; const int t = (int)(r % p.taps); const int k = (int)(r / p.taps);
        const long long src = ((long long)t * p.cout + k) * p.cin + c;
        float s = 0.f;
        for (int sp = 0; sp < p.splits; ++sp) s += p.partial[(long long)sp * n + src];
        p.out[i] = s;
    }
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* f = nullptr; cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)f;
    }
    return fn;
}

static bool encode4(CUtensorMap* m, const void* base, const uint64_t dims[4], const uint64_t strides_bytes[3], const uint32_t box[4]) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t d[4] = {dims[0], dims[1], dims[2], dims[3]};
    cuuint64_t st[3] = {strides_bytes[0], strides_bytes[1], strides_bytes[2]};
    cuuint32_t b[4] = {box[0], box[1], box[2], box[3]};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcGeom { int stages, chan_a, ncol, n_tile, kc, nchunks, Wp, box_w, box_h, plane_bytes, a_stage, b_stage, b_tap, tiles_per_img, n_img, H, W, flat, tmem_cols; size_t smem; };

// Decides whether (and how) the tensor-core kernel takes this problem.
static bool tc_geometry(const ConvProb& p, int mode, TcGeom& g) {
    if (mode == CONV_WGRAD) return false;
    // A stride-2 forward layer is computed at stride 1 and only the even positions are stored; stride-2 dgrad
    // arrives here as a stride-1 problem on a zero-stuffed dy (see zero_stuff_kernel).
    if ((p.ksz != 1 && p.ksz != 3) || p.stride < 1 || p.stride > 2 || (p.stride == 2 && mode != CONV_FWD)) return false;
    if (p.C % 16 || p.K % 16) return false;
    if (((uintptr_t)p.act | (uintptr_t)p.wgt | (uintptr_t)p.out | (uintptr_t)p.add) & 15) return false;
    g.chan_a = mode == CONV_FWD ? p.C : p.K;            // reduction channels
    g.ncol = mode == CONV_FWD ? p.K : p.C;              // output channels
    g.flat = p.ksz == 1 && p.stride == 1;
    const int taps = p.ksz * p.ksz, pad2 = p.ksz - 1;
    if (g.flat) { g.n_img = 1; g.H = 1; g.W = p.N * p.H * p.W; g.Wp = g.W; g.box_w = 128; g.box_h = 1;
        g.tiles_per_img = (int)(((long long)g.W + 127) / 128); }
    else { g.n_img = p.N; g.H = p.H; g.W = p.W; g.Wp = p.W + pad2; if (g.Wp > 128) return false;
        const int rows = (g.Wp - 1 + 127) / g.Wp + 1;   // rows 128 consecutive positions can touch
        g.box_w = g.Wp; g.box_h = std::min(rows, p.H) + pad2; if (g.box_h > 256) return false;
        g.tiles_per_img = (p.H * g.Wp + 127) / 128; }
    g.n_tile = g.ncol; while (g.n_tile > 128) { if (g.n_tile % 2) return false; g.n_tile /= 2; }
    if (g.n_tile % 16) return false;
    int kc = g.chan_a > 64 ? 64 : g.chan_a;
    while (kc > 16 && (taps * g.n_tile * kc * 2 > 80 * 1024 || g.chan_a % kc)) kc -= 16;
    if (g.chan_a % kc || taps * g.n_tile * kc * 2 > 100 * 1024) return false;
    g.kc = kc; g.nchunks = g.chan_a / kc;
    // a plane must hold the box and cover every address an MMA can touch: 128 rows past the largest tap shift
    const int max_read = (g.flat ? 0 : g.Wp - 1) + (p.ksz - 1) * g.Wp + (p.ksz - 1) + 128;
    const int plane_px = std::max(g.box_w * g.box_h, max_read);
    g.plane_bytes = ((plane_px * 16 + 127) / 128) * 128;
    g.a_stage = (kc / 8) * g.plane_bytes;
    g.b_tap = g.n_tile * kc * 2; g.b_stage = ((taps * g.b_tap + 127) / 128) * 128;
    g.stages = g.nchunks > 1 ? TC_STAGES : 1;
    g.smem = (size_t)g.stages * (g.a_stage + g.b_stage) + 256;
    if (g.smem > 200 * 1024) return false;
    g.tmem_cols = 32; while (g.tmem_cols < g.n_tile) g.tmem_cols *= 2;
    return true;
}

bool conv_tc_supported(const ConvProb& p, int mode) { TcGeom g; return encode_fn() != nullptr && tc_geometry(p, mode, g); }
size_t conv_tc_scratch_bytes(const ConvProb&, int) { return sizeof(TcProb) + 64; }

static int* g_status = nullptr;      // one status word per process, zeroed at creation
int* conv_tc_status_word() {
    if (!g_status) { cudaMalloc(&g_status, 256); cudaMemset(g_status, 0, 256); }
    return g_status;
}
int conv_tc_read_status() {
    if (!g_status) return 0;
    int v = 0; cudaMemcpy(&v, g_status, 4, cudaMemcpyDeviceToHost); return v;
}

// Fills a host-side TcProb for this problem.  Returns false when the problem is not supported.
bool conv_tc_fill(const ConvProb& p, int mode, void* host_tc) {
    TcGeom g; if (!tc_geometry(p, mode, g)) return false;
    TcProb t; memset(&t, 0, sizeof(t));
    const int taps = p.ksz * p.ksz;
    // activations: (channel, x, y, image), bf16, channels contiguous
    { const uint64_t dims[4] = {(uint64_t)g.chan_a, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.n_img};
      const uint64_t st[3] = {(uint64_t)g.chan_a * 2, (uint64_t)g.chan_a * 2 * g.W, (uint64_t)g.chan_a * 2 * g.W * g.H};
      const uint32_t box[4] = {8, (uint32_t)g.box_w, (uint32_t)g.box_h, 1};
      if (!encode4(&t.map_a, p.act, dims, st, box)) return false; }
    // weights [K][k][k][C] viewed as (8 input channels, output channel K, input-channel group C/8, tap)
    { const uint64_t dims[4] = {8, (uint64_t)p.K, (uint64_t)p.C / 8, (uint64_t)taps};
      const uint64_t st[3] = {(uint64_t)taps * p.C * 2, 16, (uint64_t)p.C * 2};
      uint32_t box[4];
      if (mode == CONV_FWD) { box[0] = 8; box[1] = g.n_tile; box[2] = g.kc / 8; box[3] = taps; }
      else { box[0] = 8; box[1] = g.kc; box[2] = g.n_tile / 8; box[3] = taps; }
      if (!encode4(&t.map_b, p.wgt, dims, st, box)) return false; }
    t.add = (const __nv_bfloat16*)p.add; t.out = (__nv_bfloat16*)p.out; t.status = conv_tc_status_word();
    t.H = g.H; t.W = g.W; t.Wp = g.Wp; t.pad = p.ksz / 2; t.taps = taps; t.flip = mode == CONV_DGRAD ? 1 : 0;
    t.n_img = g.n_img; t.tiles_per_img = g.tiles_per_img; t.tiles_n = g.ncol / g.n_tile; t.ncol = g.ncol; t.n_tile = g.n_tile;
    t.kc = g.kc; t.nchunks = g.nchunks; t.box_w = g.box_w; t.box_h = g.box_h; t.plane_bytes = g.plane_bytes;
    t.a_stage_bytes = g.a_stage; t.b_stage_bytes = g.b_stage; t.b_tap_bytes = g.b_tap; t.b_mn_major = mode == CONV_DGRAD ? 1 : 0;
    t.tmem_cols = g.tmem_cols; t.flat = g.flat; t.scale = p.scale; t.stages = g.stages;
    t.os = (mode == CONV_FWD) ? p.stride : 1; t.P = p.P; t.Q = p.Q;
    memcpy(host_tc, &t, sizeof(t));
    return true;
}
size_t conv_tc_prob_bytes() { return sizeof(TcProb); }
int conv_tc_tiles(const void* host_tc) { const TcProb* t = (const TcProb*)host_tc; return t->n_img * t->tiles_per_img * t->tiles_n; }
size_t conv_tc_smem(const void* host_tc) {
    const TcProb* t = (const TcProb*)host_tc; return (size_t)t->stages * (t->a_stage_bytes + t->b_stage_bytes) + 256;
}

void launch_conv_tc_probs(const void* d_tc, int nprob, int max_tiles, size_t max_smem, cudaStream_t s) {
    static size_t configured = 0;
    if (max_smem > configured) {
        cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(200 * 1024 + 256));
        configured = 200 * 1024 + 256;
    }
    conv_tc_kernel<<<dim3(max_tiles, nprob), TC_THREADS, max_smem, s>>>((const TcProb*)d_tc);
}

// ---- wgrad host side
struct WgGeom { int flat, n_img, H, W, Wp, tiles_per_img, pixel_tiles, m_tiles, n_tile, n_tiles, tap_groups, taps_per_group, splits,
                tiles_per_split, box_w, box_h_a, box_h_dy, plane_a, plane_dy, dy_planes, a_planes, stage_bytes, stages, tmem_cols; size_t smem, partial_bytes; };

static bool wg_geometry(const ConvProb& p, int target_ctas, WgGeom& g) {
    if (p.stride != 1 || (p.ksz != 1 && p.ksz != 3)) return false;
    if (p.C % 16 || p.K % 8) return false;
    if (p.K > 128 && p.K % 128) return false;
    if (((uintptr_t)p.act | (uintptr_t)p.wgt) & 15) return false;
    const int taps = p.ksz * p.ksz;
    g.flat = p.ksz == 1;                 // (a stride-2 1x1 layer arrives with stride 1 and a zero-stuffed dy: still flat)
    int rows = 1;
    if (g.flat) { g.n_img = 1; g.H = 1; g.W = p.N * p.H * p.W; g.Wp = g.W; g.box_w = 128; g.tiles_per_img = (int)(((long long)g.W + 127) / 128); }
    else { g.n_img = p.N; g.H = p.H; g.W = p.W; g.Wp = p.W + (p.ksz - 1); if (g.Wp > 128) return false;
        // every one of the 128 positions of a stage enters the reduction, so all of them must hold data or the
        // zero fill of the TMA box, never stale shared memory: the boxes cover every row 128 positions can touch
        // (rows past the image come back as zeros), and the activation box has one row to spare for the two
        // pixels the last tap reaches past its halo
        rows = (g.Wp - 1 + 127) / g.Wp + 1; g.box_w = g.Wp; g.tiles_per_img = (p.H * g.Wp + 127) / 128; }
    g.box_h_dy = rows; g.box_h_a = g.flat ? 1 : rows + 3;
    if (g.box_h_a > 256) return false;
    g.pixel_tiles = g.n_img * g.tiles_per_img;
    g.m_tiles = (p.K + 127) / 128;
    g.n_tile = p.C; while (g.n_tile > 256 || (g.n_tile > 64 && taps > 1 && g.n_tile * 3 > 512)) { if (g.n_tile % 32) return false; g.n_tile /= 2; }
    g.n_tiles = p.C / g.n_tile;
    g.taps_per_group = std::min(taps, 512 / g.n_tile); if (taps == 9 && g.taps_per_group < 9) g.taps_per_group = std::min(g.taps_per_group, 3);
    if (g.taps_per_group < 1) return false;
    g.tap_groups = (taps + g.taps_per_group - 1) / g.taps_per_group;
    g.tmem_cols = 32; while (g.tmem_cols < g.taps_per_group * g.n_tile) g.tmem_cols *= 2;
    if (g.tmem_cols > 512) return false;
    // planes: the MMA addresses 16 planes of dy whatever cout is; the bytes past the real planes only have to exist
    g.plane_a = ((g.box_w * g.box_h_a * 16 + 127) / 128) * 128;
    g.plane_dy = ((g.box_w * g.box_h_dy * 16 + 127) / 128) * 128;
    g.dy_planes = std::min(p.K, 128) / 8;
    g.a_planes = g.n_tile / 8;
    g.stage_bytes = g.dy_planes * g.plane_dy + g.a_planes * g.plane_a;
    const int slack = 16 * g.plane_dy + 256;
    g.stages = 4; while (g.stages > 1 && (size_t)g.stages * g.stage_bytes + slack > 200 * 1024) --g.stages;
    g.smem = (size_t)g.stages * g.stage_bytes + slack;
    if (g.smem > 200 * 1024) return false;
    const int fixed = g.m_tiles * g.n_tiles * g.tap_groups;
    int want = std::max(1, target_ctas / fixed); if (want > g.pixel_tiles) want = g.pixel_tiles; if (want > 256) want = 256;
    g.tiles_per_split = (g.pixel_tiles + want - 1) / want; g.splits = (g.pixel_tiles + g.tiles_per_split - 1) / g.tiles_per_split;
    g.partial_bytes = (size_t)g.splits * taps * p.K * p.C * 4;
    return true;
}

bool conv_wgrad_tc_supported(const ConvProb& p, int target_ctas, size_t* partial_bytes) {
    WgGeom g; if (!encode_fn() || !wg_geometry(p, target_ctas, g)) return false;
    if (partial_bytes) *partial_bytes = g.partial_bytes;
    return true;
}

// p.act = a, p.wgt = dy, p.out = dw (fp32), p.partial = workspace of at least partial_bytes
bool conv_wgrad_tc_fill(const ConvProb& p, int target_ctas, void* host_tc) {
    WgGeom g; if (!wg_geometry(p, target_ctas, g)) return false;
    TcWgradProb t; memset(&t, 0, sizeof(t));
    { const uint64_t dims[4] = {(uint64_t)p.K, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.n_img};
      const uint64_t st[3] = {(uint64_t)p.K * 2, (uint64_t)p.K * 2 * g.W, (uint64_t)p.K * 2 * g.W * g.H};
      const uint32_t box[4] = {8, (uint32_t)g.box_w, (uint32_t)g.box_h_dy, 1};
      if (!encode4(&t.map_dy, p.wgt, dims, st, box)) return false; }
    { const uint64_t dims[4] = {(uint64_t)p.C, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)g.n_img};
      const uint64_t st[3] = {(uint64_t)p.C * 2, (uint64_t)p.C * 2 * g.W, (uint64_t)p.C * 2 * g.W * g.H};
      const uint32_t box[4] = {8, (uint32_t)g.box_w, (uint32_t)g.box_h_a, 1};
      if (!encode4(&t.map_a, p.act, dims, st, box)) return false; }
    t.partial = p.partial; t.out = (float*)p.out; t.status = conv_tc_status_word();
    t.H = g.H; t.W = g.W; t.Wp = g.Wp; t.pad = p.ksz / 2; t.taps = p.ksz * p.ksz; t.ksz = p.ksz; t.flat = g.flat;
    t.n_img = g.n_img; t.tiles_per_img = g.tiles_per_img; t.pixel_tiles = g.pixel_tiles;
    t.cout = p.K; t.cin = p.C; t.m_tiles = g.m_tiles; t.n_tile = g.n_tile; t.n_tiles = g.n_tiles;
    t.tap_groups = g.tap_groups; t.taps_per_group = g.taps_per_group; t.splits = g.splits; t.tiles_per_split = g.tiles_per_split;
    t.box_w = g.box_w; t.box_h_a = g.box_h_a; t.box_h_dy = g.box_h_dy; t.plane_a = g.plane_a; t.plane_dy = g.plane_dy;
    t.dy_planes = g.dy_planes; t.a_planes = g.a_planes; t.stage_bytes = g.stage_bytes; t.stages = g.stages; t.tmem_cols = g.tmem_cols;
    memcpy(host_tc, &t, sizeof(t));
    return true;
}
size_t conv_wgrad_tc_prob_bytes() { return sizeof(TcWgradProb); }
int conv_wgrad_tc_ctas(const void* h) { const TcWgradProb* t = (const TcWgradProb*)h; return t->m_tiles * t->n_tiles * t->tap_groups * t->splits; }
size_t conv_wgrad_tc_smem(const void* h) { const TcWgradProb* t = (const TcWgradProb*)h; return (size_t)t->stages * t->stage_bytes + 16 * t->plane_dy + 256; }
long long conv_wgrad_tc_out_elems(const void* h) { const TcWgradProb* t = (const TcWgradProb*)h; return (long long)t->taps * t->cout * t->cin; }

void launch_conv_wgrad_tc_probs(const void* d_tc, int nprob, int max_ctas, size_t max_smem, long long max_out, cudaStream_t s) {
    static bool configured = false;
    if (!configured) { cudaFuncSetAttribute(conv_wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(200 * 1024 + 256)); configured = true; }
    conv_wgrad_tc_kernel<<<dim3(max_ctas, nprob), TC_THREADS, max_smem, s>>>((const TcWgradProb*)d_tc);
    long long gx = (max_out + 255) / 256; if (gx > 592) gx = 592; if (gx < 1) gx = 1;
    wgrad_tc_reduce_kernel<<<dim3((unsigned)gx, nprob), 256, 0, s>>>((const TcWgradProb*)d_tc);
}

}  // namespace resist
