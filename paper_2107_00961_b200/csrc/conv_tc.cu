// Tensor-core convolutions for sm_100a: implicit GEMM on tcgen05.mma with the accumulators in TMEM and the
// operands staged in shared memory by TMA with the 128-byte swizzle.
//
// Positions.  A 1x1 layer is a plain GEMM over the pixels of the tensor ("flat").  A 3x3 layer walks the batch as
// one tall zero-padded map: every image contributes Hp = H + 1 rows of Wp = W + 1 positions, the first row and the
// last column being zero (they are the padding of both neighbours).  In that order the operand of filter tap (r,s)
// is the SAME run of positions shifted by (r-1)*Wp + (s-1), so a tile's input window (128 positions plus a halo of
// Wp + 1 on either side) is fetched ONCE per 64-channel slab and all nine taps read it through shared-memory
// descriptors whose start address is moved by whole 128-byte rows.  The window is fetched as boxes of R tall rows
// (R divides Hp, so a box never straddles two images); the zero row and column are the out-of-bounds fill of TMA.
//
// Shared memory.  One row = one position x 64 channels = 128 bytes, rows consecutive, 16-byte chunks of a row
// XOR-swizzled with the row index (CU_TENSOR_MAP_SWIZZLE_128B writes that pattern by absolute shared-memory address
// and the tensor core reads it back by absolute address, so a descriptor may start at any 128-byte row).  Activations are K-major operands; weights are K-major in forward
// ([out channel][64 in channels]) and MN-major in dgrad ([64 reduction channels][64 out columns] blocks).
//
// Kernel structure (192 threads, one CTA per SM, persistent over the tiles of all problems of the launch):
// warp 0 = TMA producer (a ring of activation windows and a ring of weight tiles, one weight tile per (slab, tap)),
// warp 1 = TMEM owner + MMA issuer (two accumulators: the epilogue of tile i overlaps the MMAs of tile i+1),
// warps 2..5 = epilogue (TMEM -> registers -> scale, residual add, bf16 -> global).  Every wait is bounded: on expiry
// the kernel records the place in the status word, drains its copies, frees its TMEM and returns.
#include <cuda.h>
#include <cstdio>
#include <cstring>
#include <algorithm>
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
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait: false when the barrier did not flip within the limit or another role of the CTA gave up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i > 64) { __nanosleep(64); if (*abort_flag) return false; }
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(tmap), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle: start >> 4 | leading-dimension offset >> 4 at bit 16 | stride-dimension
// offset >> 4 at bit 32 | version 1 at bit 46 | swizzle mode 2 (128 bytes) at bit 61.  The base-offset field (bit 49) stays 0:
// the tensor core derives the XOR phase of a row from the row's absolute shared-memory address, exactly as TMA wrote it, so a
// start address moved by whole 128-byte rows needs nothing else (measured: with the row phase in the field the taps read the
// wrong 16-byte chunks).
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                   "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]),
                   "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]),
                   "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr));
}
__device__ __forceinline__ int floor_div(int a, int b) { int q = a / b; if ((a % b != 0) && ((a < 0) != (b < 0))) --q; return q; }

constexpr int TC_THREADS = 192;
constexpr int TC_MAX_STAGES = 6;
constexpr int TILE_M = 128;

// One forward / dgrad problem.  The two tensor maps come first so that each is 64-byte aligned.
struct alignas(64) TcProb {
    CUtensorMap map_a;        // activations (forward: a; dgrad: dy): flat (channel, pixel); tall (channel, x, y, image)
    CUtensorMap map_b;        // weights [K][taps][C] viewed as (C, tap, K)
    const __nv_bfloat16* add; __nv_bfloat16* out;
    int* status;
    int flat, taps, ksz, flip;               // flip: dgrad reads weight tap taps-1-t for window tap t
    int H, W, Wp, Hp, n_img;
    int R, box_pos, nbox, halo;              // window = nbox boxes of R tall rows (box_pos positions each); halo = Wp + 1 or 0
    int a_box_bytes;
    int tiles_m, tiles_n, n_tile, ncol;      // output tile grid; MMA N; channels of the output tensor
    int red, slabs;                          // reduction channels, 64-channel slabs
    int b_mn_major;                          // 0: forward (weights K-major); 1: dgrad (weights MN-major)
    int b_bytes;                             // bytes of one weight tile (one slab, one tap)
    long long total_pos;                     // positions walked (flat: pixels; tall: n_img * Hp * Wp)
    float scale;
    int os, P, Q;                            // output stride: only positions (y, x) with y, x multiples of os are stored, as pixel (y/os, x/os) of a P x Q image
};

struct TcLaunch { int nprob, na, nb, a_stage, b_stage, tmem_cols, acc_stride; };

__global__ void __launch_bounds__(TC_THREADS, 1) conv_tc_kernel(const TcProb* __restrict__ probs, const TcLaunch L) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[4 * TC_MAX_STAGES + 4];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    const uint32_t a_full = smem_u32(&bars[0]), a_empty = smem_u32(&bars[TC_MAX_STAGES]);
    const uint32_t b_full = smem_u32(&bars[2 * TC_MAX_STAGES]), b_empty = smem_u32(&bars[3 * TC_MAX_STAGES]);
    const uint32_t acc_full = smem_u32(&bars[4 * TC_MAX_STAGES]), acc_empty = smem_u32(&bars[4 * TC_MAX_STAGES + 2]);
    const uint32_t a_ring = smem_u32(smem), b_ring = a_ring + (uint32_t)(L.na * L.a_stage);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) {
            mbar_init(a_full + 8 * s, 1); mbar_init(a_empty + 8 * s, 1); mbar_init(b_full + 8 * s, 1); mbar_init(b_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full + 8 * s, 1); mbar_init(acc_empty + 8 * s, 4); }
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(L.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;

    int total_tiles = 0;
    for (int i = 0; i < L.nprob; ++i) total_tiles += probs[i].tiles_m * probs[i].tiles_n;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t a_cnt = 0, b_cnt = 0; bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                int pi = 0, loc = t;
                while (loc >= probs[pi].tiles_m * probs[pi].tiles_n) { loc -= probs[pi].tiles_m * probs[pi].tiles_n; ++pi; }
                const TcProb& p = probs[pi];
                const int tn = loc % p.tiles_n, tm = loc / p.tiles_n;
                const int bx0 = p.flat ? 0 : floor_div(tm * TILE_M - p.halo, p.box_pos);
                for (int sl = 0; sl < p.slabs && ok; ++sl) {
                    {
                        const int s = (int)(a_cnt % (uint32_t)L.na); const uint32_t ph = (a_cnt / (uint32_t)L.na) & 1u;
                        if (!mbar_wait(a_empty + 8 * s, ph ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 1); ok = false; break; }
                        const uint32_t dst = a_ring + (uint32_t)(s * L.a_stage);
                        mbar_expect_tx(a_full + 8 * s, (uint32_t)(p.nbox * p.a_box_bytes));
                        if (p.flat) tma_load_2d(dst, &p.map_a, a_full + 8 * s, sl * 64, tm * TILE_M);
                        else for (int i = 0; i < p.nbox; ++i) {
                            const int trow = (bx0 + i) * p.R, img = floor_div(trow, p.Hp), y0 = trow - img * p.Hp - 1;
                            tma_load_4d(dst + (uint32_t)(i * p.a_box_bytes), &p.map_a, a_full + 8 * s, sl * 64, 0, y0, img);
                        }
                        ++a_cnt;
                    }
                    for (int tap = 0; tap < p.taps; ++tap) {
                        const int s = (int)(b_cnt % (uint32_t)L.nb); const uint32_t ph = (b_cnt / (uint32_t)L.nb) & 1u;
                        if (!mbar_wait(b_empty + 8 * s, ph ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 2); ok = false; break; }
                        const uint32_t dst = b_ring + (uint32_t)(s * L.b_stage);
                        const int wtap = p.flip ? p.taps - 1 - tap : tap;
                        mbar_expect_tx(b_full + 8 * s, (uint32_t)p.b_bytes);
                        if (!p.b_mn_major) tma_load_3d(dst, &p.map_b, b_full + 8 * s, sl * 64, wtap, tn * p.n_tile);
                        else for (int j = 0; j * 64 < p.n_tile; ++j)
                            tma_load_3d(dst + (uint32_t)(j * 8192), &p.map_b, b_full + 8 * s, tn * p.n_tile + j * 64, wtap, sl * 64);
                        ++b_cnt;
                    }
                }
            }
            if (!ok) {
                // another role gave up (or this one): wait, bounded, for the copies still in flight before the CTA leaves
                for (uint32_t c = a_cnt > (uint32_t)L.na ? a_cnt - L.na : 0; c < a_cnt; ++c)
                    for (int i = 0; i < 4096 && !mbar_try(a_full + 8 * (c % L.na), (c / L.na) & 1u); ++i) __nanosleep(64);
                for (uint32_t c = b_cnt > (uint32_t)L.nb ? b_cnt - L.nb : 0; c < b_cnt; ++c)
                    for (int i = 0; i < 4096 && !mbar_try(b_full + 8 * (c % L.nb), (c / L.nb) & 1u); ++i) __nanosleep(64);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t a_cnt = 0, b_cnt = 0, acc_cnt = 0; bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++acc_cnt) {
                int pi = 0, loc = t;
                while (loc >= probs[pi].tiles_m * probs[pi].tiles_n) { loc -= probs[pi].tiles_m * probs[pi].tiles_n; ++pi; }
                const TcProb& p = probs[pi];
                const int tm = loc / p.tiles_n;
                const int bx0 = p.flat ? 0 : floor_div(tm * TILE_M - p.halo, p.box_pos);
                const int a_off = p.flat ? 0 : tm * TILE_M - p.halo - bx0 * p.box_pos;
                const uint32_t buf = acc_cnt & 1u, aph = (acc_cnt >> 1) & 1u;
                if (!mbar_wait(acc_empty + 8 * buf, aph ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 3); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)L.acc_stride;
                // instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B K-major or MN-major, N, M = 128
                const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.b_mn_major << 16) |
                                       ((uint32_t)(p.n_tile >> 3) << 17) | ((128u >> 4) << 24);
                uint32_t acc = 0;
                for (int sl = 0; sl < p.slabs && ok; ++sl) {
                    const int sa = (int)(a_cnt % (uint32_t)L.na); const uint32_t pha = (a_cnt / (uint32_t)L.na) & 1u;
                    if (!mbar_wait(a_full + 8 * sa, pha, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 4); ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_base = a_ring + (uint32_t)(sa * L.a_stage) + (uint32_t)a_off * 128u;
                    const int ksteps = (min(64, p.red - sl * 64) + 15) >> 4;
                    for (int tap = 0; tap < p.taps; ++tap) {
                        const int sb = (int)(b_cnt % (uint32_t)L.nb); const uint32_t phb = (b_cnt / (uint32_t)L.nb) & 1u;
                        if (!mbar_wait(b_full + 8 * sb, phb, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 5); ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const int r = tap / p.ksz, q = tap - r * p.ksz;
                        const uint32_t a_tap = a_base + (uint32_t)(r * p.Wp + q) * 128u;
                        const uint32_t b_base = b_ring + (uint32_t)(sb * L.b_stage);
                        for (int k16 = 0; k16 < ksteps; ++k16) {
                            const uint64_t ad = desc_sw128(a_tap + (uint32_t)k16 * 32u, 16, 1024);
                            const uint64_t bd = p.b_mn_major ? desc_sw128(b_base + (uint32_t)k16 * 2048u, 8192, 1024)
                                                             : desc_sw128(b_base + (uint32_t)k16 * 32u, 16, 1024);
                            umma_bf16(d_tmem, ad, bd, idesc, acc);
                            acc = 1;
                        }
                        umma_commit(b_empty + 8 * sb);           // weight tile reusable once these MMAs have read it
                        ++b_cnt;
                    }
                    umma_commit(a_empty + 8 * sa);
                    ++a_cnt;
                }
                if (ok) umma_commit(acc_full + 8 * buf);         // accumulator complete
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue: 4 warps, one TMEM lane quadrant each
        const int quad = warp & 3;
        const int m = quad * 32 + lane;                          // row of the tile = TMEM lane
        uint32_t acc_cnt = 0; bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++acc_cnt) {
            int pi = 0, loc = t;
            while (loc >= probs[pi].tiles_m * probs[pi].tiles_n) { loc -= probs[pi].tiles_m * probs[pi].tiles_n; ++pi; }
            const TcProb& p = probs[pi];
            const int tn = loc % p.tiles_n, tm = loc / p.tiles_n;
            const uint32_t buf = acc_cnt & 1u, aph = (acc_cnt >> 1) & 1u;
            ok = mbar_wait(acc_full + 8 * buf, aph, &abort_s);
            ok = __all_sync(0xffffffffu, ok);                    // tcgen05.ld below is warp-collective
            if (!ok) { atomicExch(&abort_s, 1); atomicExch(p.status, 6); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // position -> output pixel
            long long pix = -1;
            const long long pos = (long long)tm * TILE_M + m;
            if (p.flat) { if (pos < p.total_pos) pix = pos; }
            else if (pos < p.total_pos) {
                const int trow = (int)(pos / p.Wp), x = (int)(pos - (long long)trow * p.Wp);
                const int img = trow / p.Hp, y = trow - img * p.Hp - 1;
                if (x < p.W && y >= 0) {
                    if (p.os == 1) pix = ((long long)img * p.H + y) * p.W + x;
                    else if (y % p.os == 0 && x % p.os == 0) pix = ((long long)img * p.P + y / p.os) * p.Q + x / p.os;   // strided layer
                }
            }
            const uint32_t t_row = tmem_base + buf * (uint32_t)L.acc_stride + ((uint32_t)(quad * 32) << 16);
            const int col0 = tn * p.n_tile;
            for (int c0 = 0; c0 < p.n_tile; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(t_row + (uint32_t)c0, v);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (pix >= 0) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const int c = c0 + g * 8;
                        if (c < p.n_tile && col0 + c < p.ncol) {
                            const long long o = pix * p.ncol + col0 + c;
                            float f[8];
#pragma unroll
                            for (int k = 0; k < 8; ++k) f[k] = __uint_as_float(v[g * 8 + k]) * p.scale;
                            if (p.add) {
                                const uint4 a0 = *reinterpret_cast<const uint4*>(p.add + o);
                                const uint32_t aw[4] = {a0.x, a0.y, a0.z, a0.w};
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    f[2 * k] += __uint_as_float(aw[k] << 16);
                                    f[2 * k + 1] += __uint_as_float(aw[k] & 0xFFFF0000u);
                                }
                            }
                            uint32_t w[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
                                w[k] = *reinterpret_cast<uint32_t*>(&h);
                            }
                            *reinterpret_cast<uint4*>(p.out + o) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty + 8 * buf);     // this warp has read its quadrant of the accumulator
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(L.tmem_cols) : "memory");
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
// dw[k][r][s][c] = sum over output positions of dy[pos][k] * a[pos + shift(r,s)][c].  The reduction runs over the
// positions of the forward kernel (flat pixels, or the tall zero-padded map, where dy reads as zero at the padding
// positions and adds nothing), 128 per pipeline stage: D[cout (128 lanes), cin] per tap, A = dy^T and B = shifted a,
// both MN-major straight from their 128-byte rows.  A CTA accumulates a range of position chunks for a group of taps
// and writes an fp32 partial (or, alone on its tile, the result); a second kernel adds the partials in a fixed order.
struct alignas(64) TcWgradProb {
    CUtensorMap map_dy;       // flat (channel k, pixel); tall (channel k, x, y, image)
    CUtensorMap map_a;        // likewise for a
    float* partial;           // [splits][taps][cout][cin]
    float* out;               // [cout][taps][cin]
    int* status;
    int flat, taps, ksz;
    int H, W, Wp, Hp, n_img;
    int R, box_pos, nbox_dy, nbox_a, halo, box_bytes;
    int chunks;                                   // position chunks of 128 in total
    int cout, cin, m_tiles, n_tile, n_tiles, a_slabs;
    int tap_groups, taps_per_group, splits, chunks_per_split;
    int dy_slab_bytes, a_slab_bytes;              // one 64-channel slab of a stage
    int stage_bytes, stages, tmem_cols;
};

__global__ void __launch_bounds__(TC_THREADS, 1) conv_wgrad_tc_kernel(const TcWgradProb* __restrict__ probs) {
    const TcWgradProb& p = probs[blockIdx.y];
    const int ctas = p.m_tiles * p.n_tiles * p.tap_groups * p.splits;
    if ((int)blockIdx.x >= ctas) return;
    int id = blockIdx.x;
    const int split = id % p.splits; id /= p.splits;
    const int tg = id % p.tap_groups; id /= p.tap_groups;
    const int tn = id % p.n_tiles; const int tm = id / p.n_tiles;
    const int c_begin = split * p.chunks_per_split;
    const int c_end = min(c_begin + p.chunks_per_split, p.chunks);
    const int tap0 = tg * p.taps_per_group;
    const int ntap = min(p.taps - tap0, p.taps_per_group);
    const int nc = c_end - c_begin;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[2 * TC_MAX_STAGES + 1];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[TC_MAX_STAGES]), bar_acc = smem_u32(&bars[2 * TC_MAX_STAGES]);
    const uint32_t ring = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
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
        if (lane == 0) {
            int i = 0; bool ok = true;
            for (; i < nc; ++i) {
                const int s = i % p.stages; const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
                if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 11); ok = false; break; }
                const int pos0 = (c_begin + i) * TILE_M;
                const uint32_t dy_dst = ring + (uint32_t)(s * p.stage_bytes), a_dst = dy_dst + 2u * (uint32_t)p.dy_slab_bytes;
                mbar_expect_tx(bar_full + 8 * s, (uint32_t)((2 * p.nbox_dy + p.a_slabs * p.nbox_a) * p.box_bytes));
                if (p.flat) {
                    for (int j = 0; j < 2; ++j) tma_load_2d(dy_dst + (uint32_t)(j * p.dy_slab_bytes), &p.map_dy, bar_full + 8 * s, tm * 128 + j * 64, pos0);
                    for (int j = 0; j < p.a_slabs; ++j) tma_load_2d(a_dst + (uint32_t)(j * p.a_slab_bytes), &p.map_a, bar_full + 8 * s, tn * p.n_tile + j * 64, pos0);
                } else {
                    const int bd0 = pos0 / p.box_pos, ba0 = floor_div(pos0 - p.halo, p.box_pos);
                    for (int b = 0; b < p.nbox_dy; ++b) {
                        const int trow = (bd0 + b) * p.R, img = trow / p.Hp, y0 = trow - img * p.Hp - 1;
                        for (int j = 0; j < 2; ++j)
                            tma_load_4d(dy_dst + (uint32_t)(j * p.dy_slab_bytes + b * p.box_bytes), &p.map_dy, bar_full + 8 * s, tm * 128 + j * 64, 0, y0, img);
                    }
                    for (int b = 0; b < p.nbox_a; ++b) {
                        const int trow = (ba0 + b) * p.R, img = floor_div(trow, p.Hp), y0 = trow - img * p.Hp - 1;
                        for (int j = 0; j < p.a_slabs; ++j)
                            tma_load_4d(a_dst + (uint32_t)(j * p.a_slab_bytes + b * p.box_bytes), &p.map_a, bar_full + 8 * s, tn * p.n_tile + j * 64, 0, y0, img);
                    }
                }
            }
            if (!ok)
                for (int c = max(0, i - p.stages); c < i; ++c)
                    for (int w = 0; w < 4096 && !mbar_try(bar_full + 8 * (c % p.stages), (uint32_t)(c / p.stages) & 1u); ++w) __nanosleep(64);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // fp32 accumulate, bf16 x bf16, A and B MN-major, N = n_tile, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(p.n_tile >> 3) << 17) | ((128u >> 4) << 24);
            bool ok = true;
            for (int i = 0; i < nc && ok; ++i) {
                const int s = i % p.stages; const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
                if (!mbar_wait(bar_full + 8 * s, ph, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 12); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int pos0 = (c_begin + i) * TILE_M;
                int dy_off = 0, a_off = 0;
                if (!p.flat) { dy_off = pos0 - (pos0 / p.box_pos) * p.box_pos; a_off = pos0 - p.halo - floor_div(pos0 - p.halo, p.box_pos) * p.box_pos; }
                const uint32_t dy_base = ring + (uint32_t)(s * p.stage_bytes) + (uint32_t)dy_off * 128u;
                const uint32_t a_base = ring + (uint32_t)(s * p.stage_bytes) + 2u * (uint32_t)p.dy_slab_bytes + (uint32_t)a_off * 128u;
                for (int tt = 0; tt < ntap; ++tt) {
                    const int t = tap0 + tt, r = t / p.ksz, q = t - r * p.ksz;
                    const uint32_t a_tap = a_base + (uint32_t)(r * p.Wp + q) * 128u;
                    for (int k16 = 0; k16 < 8; ++k16) {
                        const uint64_t ad = desc_sw128(dy_base + (uint32_t)k16 * 2048u, (uint32_t)p.dy_slab_bytes, 1024);
                        const uint64_t bd = desc_sw128(a_tap + (uint32_t)k16 * 2048u, (uint32_t)p.a_slab_bytes, 1024);
                        umma_bf16(tmem_d + (uint32_t)(tt * p.n_tile), ad, bd, idesc, (i | k16) ? 1u : 0u);
                    }
                }
                umma_commit(bar_empty + 8 * s);
            }
            if (ok) umma_commit(bar_acc);
        }
    } else {
        const int quad = warp & 3, m = quad * 32 + lane;
        bool ok = nc > 0 ? mbar_wait(bar_acc, 0, &abort_s) : true;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { atomicExch(&abort_s, 1); atomicExch(p.status, 13); }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int k = tm * 128 + m;
        if (ok && quad * 32 < p.cout - tm * 128) {            // warp-uniform: this lane quadrant holds real output channels
            for (int tt = 0; tt < ntap; ++tt) {
                float* dst = p.splits > 1 ? p.partial + (((long long)split * p.taps + tap0 + tt) * p.cout + k) * p.cin + tn * p.n_tile
                                          : p.out + ((long long)k * p.taps + tap0 + tt) * p.cin + tn * p.n_tile;
                for (int c0 = 0; c0 < p.n_tile; c0 += 32) {
                    uint32_t v[32];
                    if (nc > 0) { tmem_ld32(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(tt * p.n_tile + c0), v);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
                    else { for (int j = 0; j < 32; ++j) v[j] = 0u; }
                    if (k < p.cout) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (c0 + j < p.n_tile && tn * p.n_tile + c0 + j < p.cin)
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
    if (p.splits <= 1) return;                                 // the convolution kernel wrote the result itself
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

// bf16 tensor map of `rank` dimensions (innermost first), 128-byte swizzle, zero fill out of bounds
static bool encode_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t d[5]; cuuint64_t st[4]; cuuint32_t b[5]; cuuint32_t es[5];
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; if (i + 1 < rank) st[i] = strides_bytes[i]; }
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// activations [n_img][H][W][chan] as the tall map's source (channel, x, y, image), or flat (channel, pixel)
static bool encode_act(CUtensorMap* m, const void* base, int chan, bool flat, long long pixels, int n_img, int H, int W, int Wp, int R) {
    if (flat) {
        const uint64_t dims[2] = {(uint64_t)chan, (uint64_t)pixels}; const uint64_t st[1] = {(uint64_t)chan * 2}; const uint32_t box[2] = {64, 128};
        return encode_map(m, base, 2, dims, st, box);
    }
    const uint64_t dims[4] = {(uint64_t)chan, (uint64_t)W, (uint64_t)H, (uint64_t)n_img};
    const uint64_t st[3] = {(uint64_t)chan * 2, (uint64_t)chan * 2 * W, (uint64_t)chan * 2 * W * H};
    const uint32_t box[4] = {64, (uint32_t)Wp, (uint32_t)R, 1};
    return encode_map(m, base, 4, dims, st, box);
}

// rows of the tall map fetched by one box: the largest divisor of Hp whose box holds at most 64 positions
static int box_rows(int Hp, int Wp) { int best = 1; for (int r = 1; r <= Hp; ++r) if (Hp % r == 0 && r * Wp <= 64) best = r; return best; }

struct TcGeom { int flat, chan_a, ncol, n_tile, tiles_n, tiles_m, slabs, Wp, Hp, R, box_pos, nbox, halo, a_box_bytes, a_stage, b_bytes, b_stage, n_img, H, W;
                long long total_pos; };

// Decides whether (and how) the tensor-core kernel takes this problem.
static bool tc_geometry(const ConvProb& p, int mode, TcGeom& g) {
    if (mode == CONV_WGRAD) return false;
    // A stride-2 forward layer is computed at stride 1 and only the even positions are stored; stride-2 dgrad
    // arrives here as a stride-1 problem on a zero-stuffed dy (see zero_stuff_kernel).
    if ((p.ksz != 1 && p.ksz != 3) || p.stride < 1 || p.stride > 2 || (p.stride == 2 && mode != CONV_FWD)) return false;
    if (p.C % 8 || p.K % 8) return false;
    if (((uintptr_t)p.act | (uintptr_t)p.wgt | (uintptr_t)p.out | (uintptr_t)p.add) & 15) return false;
    g.chan_a = mode == CONV_FWD ? p.C : p.K;            // reduction channels
    g.ncol = mode == CONV_FWD ? p.K : p.C;              // output channels
    g.flat = p.ksz == 1 && p.stride == 1;
    g.n_img = p.N; g.H = p.H; g.W = p.W;
    if (g.flat) { g.total_pos = (long long)p.N * p.H * p.W; g.Wp = 0; g.Hp = 0; g.R = 0; g.box_pos = 128; g.nbox = 1; g.halo = 0; g.a_box_bytes = 128 * 128; }
    else {
        g.Wp = p.W + 1; g.Hp = p.H + 1; if (g.Wp > 256) return false;
        g.total_pos = (long long)p.N * g.Hp * g.Wp;
        g.R = box_rows(g.Hp, g.Wp); g.box_pos = g.R * g.Wp; g.halo = p.ksz == 3 ? g.Wp + 1 : 0;
        g.nbox = (TILE_M + 2 * g.halo + g.box_pos - 1 + g.box_pos - 1) / g.box_pos;
        g.a_box_bytes = g.box_pos * 128;
    }
    if (g.total_pos > (1ll << 30)) return false;
    g.tiles_m = (int)((g.total_pos + TILE_M - 1) / TILE_M);
    g.tiles_n = (g.ncol + 255) / 256;
    g.n_tile = (((g.ncol + g.tiles_n - 1) / g.tiles_n) + 15) / 16 * 16;
    g.slabs = (g.chan_a + 63) / 64;
    g.a_stage = (g.nbox * g.a_box_bytes + 1023) / 1024 * 1024;
    g.b_bytes = mode == CONV_FWD ? g.n_tile * 128 : ((g.n_tile + 63) / 64) * 8192;
    g.b_stage = (g.b_bytes + 1023) / 1024 * 1024;
    return true;
}

bool conv_tc_supported(const ConvProb& p, int mode) { TcGeom g; return encode_fn() != nullptr && tc_geometry(p, mode, g); }

static int* g_status = nullptr;      // one status word per process, zeroed at creation
int* conv_tc_status_word() {
    if (!g_status) { cudaMalloc(&g_status, 256); cudaMemset(g_status, 0, 256); }
    return g_status;
}
int conv_tc_read_status() {
    if (!g_status) return 0;
    int v = 0; cudaMemcpy(&v, g_status, 4, cudaMemcpyDeviceToHost);
    if (v) cudaMemset(g_status, 0, 4);              // reported once
    return v;
}

// Fills a host-side TcProb for this problem.  Returns false when the problem is not supported.
bool conv_tc_fill(const ConvProb& p, int mode, void* host_tc) {
    TcGeom g; if (!tc_geometry(p, mode, g)) return false;
    TcProb t; memset(&t, 0, sizeof(t));
    const int taps = p.ksz * p.ksz;
    if (!encode_act(&t.map_a, p.act, g.chan_a, g.flat != 0, g.total_pos, g.n_img, g.H, g.W, g.Wp, g.R)) return false;
    // weights [K][taps][C] viewed as (C, tap, K).  Forward: a tile is n_tile output channels (rows) x 64 input channels.
    // dgrad: a block is 64 reduction channels k (rows) x 64 output columns c.
    { const uint64_t dims[3] = {(uint64_t)p.C, (uint64_t)taps, (uint64_t)p.K};
      const uint64_t st[2] = {(uint64_t)p.C * 2, (uint64_t)taps * p.C * 2};
      const uint32_t box[3] = {64, 1, mode == CONV_FWD ? (uint32_t)g.n_tile : 64u};
      if (!encode_map(&t.map_b, p.wgt, 3, dims, st, box)) return false; }
    t.add = (const __nv_bfloat16*)p.add; t.out = (__nv_bfloat16*)p.out; t.status = conv_tc_status_word();
    t.flat = g.flat; t.taps = taps; t.ksz = p.ksz; t.flip = mode == CONV_DGRAD ? 1 : 0;
    t.H = g.H; t.W = g.W; t.Wp = g.Wp; t.Hp = g.Hp; t.n_img = g.n_img;
    t.R = g.R; t.box_pos = g.box_pos; t.nbox = g.nbox; t.halo = g.halo; t.a_box_bytes = g.a_box_bytes;
    t.tiles_m = g.tiles_m; t.tiles_n = g.tiles_n; t.n_tile = g.n_tile; t.ncol = g.ncol;
    t.red = g.chan_a; t.slabs = g.slabs; t.b_mn_major = mode == CONV_DGRAD ? 1 : 0; t.b_bytes = g.b_bytes;
    t.total_pos = g.total_pos; t.scale = p.scale;
    t.os = (mode == CONV_FWD) ? p.stride : 1; t.P = p.P; t.Q = p.Q;
    memcpy(host_tc, &t, sizeof(t));
    return true;
}
size_t conv_tc_prob_bytes() { return sizeof(TcProb); }
int conv_tc_tiles(const void* host_tc) { const TcProb* t = (const TcProb*)host_tc; return t->tiles_m * t->tiles_n; }
// packs what a launch has to know about its largest problem into one number: window bytes, weight-tile bytes, MMA N
size_t conv_tc_smem(const void* host_tc) {
    const TcProb* t = (const TcProb*)host_tc;
    const size_t a_stage = ((size_t)t->nbox * t->a_box_bytes + 1023) / 1024, b_stage = ((size_t)t->b_bytes + 1023) / 1024;
    return (a_stage << 40) | (b_stage << 20) | (size_t)t->n_tile;
}

// field-wise maximum of two packed values
size_t conv_tc_merge(size_t a, size_t b) {
    const size_t m20 = 0xFFFFF;
    return (std::max(a >> 40, b >> 40) << 40) | (std::max((a >> 20) & m20, (b >> 20) & m20) << 20) | std::max(a & m20, b & m20);
}

constexpr size_t TC_SMEM_BUDGET = 200 * 1024;

// total_tiles: tiles of all problems of the launch; packed: the largest conv_tc_smem() value of its problems (fields are maxima)
void launch_conv_tc_probs(const void* d_tc, int nprob, int max_tiles, size_t packed, cudaStream_t s) {
    static bool configured = false; static int sms = 0;
    if (!configured) {
        cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(TC_SMEM_BUDGET + 1024));
        int dev = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        configured = true;
    }
    TcLaunch L{};
    L.nprob = nprob;
    L.a_stage = (int)(packed >> 40) * 1024; L.b_stage = (int)((packed >> 20) & 0xFFFFF) * 1024;
    const int n_tile = (int)(packed & 0xFFFFF);
    // ring depths: up to 4 windows and up to 6 weight tiles within the budget, at least 2 of each
    L.na = 2; L.nb = 2;
    while (true) {
        bool grown = false;
        if (L.nb < TC_MAX_STAGES && (size_t)L.na * L.a_stage + (size_t)(L.nb + 1) * L.b_stage <= TC_SMEM_BUDGET) { ++L.nb; grown = true; }
        if (L.na < 4 && (size_t)(L.na + 1) * L.a_stage + (size_t)L.nb * L.b_stage <= TC_SMEM_BUDGET) { ++L.na; grown = true; }
        if (!grown) break;
    }
    L.acc_stride = (n_tile + 31) / 32 * 32;
    L.tmem_cols = 32; while (L.tmem_cols < 2 * L.acc_stride) L.tmem_cols *= 2;
    // at least 120 KB of shared memory so that two CTAs that allocate tensor memory never share an SM
    const size_t smem = std::max((size_t)L.na * L.a_stage + (size_t)L.nb * L.b_stage, (size_t)120 * 1024) + 1024;
    const int total = max_tiles * nprob;
    const int grid = std::max(1, std::min(total, sms));
    conv_tc_kernel<<<grid, TC_THREADS, smem, s>>>((const TcProb*)d_tc, L);
}

// ---- wgrad host side
struct WgGeom { int flat, n_img, H, W, Wp, Hp, R, box_pos, nbox_dy, nbox_a, halo, box_bytes, chunks, m_tiles, n_tile, n_tiles, a_slabs, tap_groups, taps_per_group,
                splits, chunks_per_split, dy_slab, a_slab, stage_bytes, stages, tmem_cols; size_t smem, partial_bytes; };

static bool wg_geometry(const ConvProb& p, int target_ctas, WgGeom& g) {
    if (p.stride != 1 || (p.ksz != 1 && p.ksz != 3)) return false;
    if (p.C % 8 || p.K % 8) return false;
    if (((uintptr_t)p.act | (uintptr_t)p.wgt) & 15) return false;
    const int taps = p.ksz * p.ksz;
    g.flat = p.ksz == 1;                 // (a stride-2 1x1 layer arrives with stride 1 and a zero-stuffed dy: still flat)
    g.n_img = p.N; g.H = p.H; g.W = p.W;
    long long total_pos;
    if (g.flat) { total_pos = (long long)p.N * p.H * p.W; g.Wp = 0; g.Hp = 0; g.R = 0; g.box_pos = 128; g.nbox_dy = 1; g.nbox_a = 1; g.halo = 0; g.box_bytes = 128 * 128; }
    else {
        g.Wp = p.W + 1; g.Hp = p.H + 1; if (g.Wp > 256) return false;
        total_pos = (long long)p.N * g.Hp * g.Wp;
        g.R = box_rows(g.Hp, g.Wp); g.box_pos = g.R * g.Wp; g.halo = g.Wp + 1; g.box_bytes = g.box_pos * 128;
        g.nbox_dy = (TILE_M + g.box_pos - 1 + g.box_pos - 1) / g.box_pos;
        g.nbox_a = (TILE_M + 2 * g.halo + g.box_pos - 1 + g.box_pos - 1) / g.box_pos;
    }
    if (total_pos > (1ll << 30)) return false;
    g.chunks = (int)((total_pos + TILE_M - 1) / TILE_M);
    g.m_tiles = (p.K + 127) / 128;
    // columns of one CTA: the input channels in tiles of at most 256 (1x1) or 128 (3x3, three taps per CTA), tap groups within 512 columns of tensor memory
    const int n_cap = taps == 1 ? 256 : 128;
    g.n_tiles = (p.C + n_cap - 1) / n_cap;
    g.n_tile = (((p.C + g.n_tiles - 1) / g.n_tiles) + 15) / 16 * 16;
    g.a_slabs = (g.n_tile + 63) / 64;
    g.taps_per_group = taps == 1 ? 1 : std::min(3, 512 / g.n_tile);
    g.tap_groups = (taps + g.taps_per_group - 1) / g.taps_per_group;
    g.tmem_cols = 32; while (g.tmem_cols < g.taps_per_group * g.n_tile) g.tmem_cols *= 2;
    if (g.tmem_cols > 512) return false;
    g.dy_slab = (g.nbox_dy * g.box_bytes + 1023) / 1024 * 1024;
    g.a_slab = (g.nbox_a * g.box_bytes + 1023) / 1024 * 1024;
    g.stage_bytes = 2 * g.dy_slab + g.a_slabs * g.a_slab;
    g.stages = TC_MAX_STAGES; while (g.stages > 1 && (size_t)g.stages * g.stage_bytes > TC_SMEM_BUDGET) --g.stages;
    if ((size_t)g.stages * g.stage_bytes > TC_SMEM_BUDGET) return false;
    g.smem = std::max((size_t)g.stages * g.stage_bytes, (size_t)120 * 1024) + 1024;
    const int fixed = g.m_tiles * g.n_tiles * g.tap_groups;
    int want = std::max(1, target_ctas / fixed); if (want > g.chunks) want = g.chunks; if (want > 256) want = 256;
    g.chunks_per_split = (g.chunks + want - 1) / want; g.splits = (g.chunks + g.chunks_per_split - 1) / g.chunks_per_split;
    g.partial_bytes = g.splits > 1 ? (size_t)g.splits * taps * p.K * p.C * 4 : 0;
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
    const long long pixels = (long long)p.N * p.H * p.W;
    if (!encode_act(&t.map_dy, p.wgt, p.K, g.flat != 0, pixels, g.n_img, g.H, g.W, g.Wp, g.R)) return false;
    if (!encode_act(&t.map_a, p.act, p.C, g.flat != 0, pixels, g.n_img, g.H, g.W, g.Wp, g.R)) return false;
    t.partial = p.partial; t.out = (float*)p.out; t.status = conv_tc_status_word();
    t.flat = g.flat; t.taps = p.ksz * p.ksz; t.ksz = p.ksz;
    t.H = g.H; t.W = g.W; t.Wp = g.Wp; t.Hp = g.Hp; t.n_img = g.n_img;
    t.R = g.R; t.box_pos = g.box_pos; t.nbox_dy = g.nbox_dy; t.nbox_a = g.nbox_a; t.halo = g.halo; t.box_bytes = g.box_bytes;
    t.chunks = g.chunks; t.cout = p.K; t.cin = p.C; t.m_tiles = g.m_tiles; t.n_tile = g.n_tile; t.n_tiles = g.n_tiles; t.a_slabs = g.a_slabs;
    t.tap_groups = g.tap_groups; t.taps_per_group = g.taps_per_group; t.splits = g.splits; t.chunks_per_split = g.chunks_per_split;
    t.dy_slab_bytes = g.dy_slab; t.a_slab_bytes = g.a_slab; t.stage_bytes = g.stage_bytes; t.stages = g.stages; t.tmem_cols = g.tmem_cols;
    memcpy(host_tc, &t, sizeof(t));
    return true;
}
size_t conv_wgrad_tc_prob_bytes() { return sizeof(TcWgradProb); }
int conv_wgrad_tc_ctas(const void* h) { const TcWgradProb* t = (const TcWgradProb*)h; return t->m_tiles * t->n_tiles * t->tap_groups * t->splits; }
size_t conv_wgrad_tc_smem(const void* h) { const TcWgradProb* t = (const TcWgradProb*)h; return std::max((size_t)t->stages * t->stage_bytes, (size_t)120 * 1024) + 1024; }
long long conv_wgrad_tc_out_elems(const void* h) { const TcWgradProb* t = (const TcWgradProb*)h; return (long long)t->taps * t->cout * t->cin; }

void launch_conv_wgrad_tc_probs(const void* d_tc, int nprob, int max_ctas, size_t max_smem, long long max_out, cudaStream_t s) {
    static bool configured = false;
    if (!configured) { cudaFuncSetAttribute(conv_wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(TC_SMEM_BUDGET + 1024)); configured = true; }
    conv_wgrad_tc_kernel<<<dim3(max_ctas, nprob), TC_THREADS, max_smem, s>>>((const TcWgradProb*)d_tc);
    long long gx = (max_out + 255) / 256; if (gx > 592) gx = 592; if (gx < 1) gx = 1;
    wgrad_tc_reduce_kernel<<<dim3((unsigned)gx, nprob), 256, 0, s>>>((const TcWgradProb*)d_tc);
}

}  // namespace resist
