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
// Kernel structure of forward / dgrad (352 threads, one CTA per SM, persistent over the work of all problems of the launch).  A
// unit of work is a PAIR of neighbouring 128-position tiles times one column tile of up to 256 output channels:
// warp 0 = TMA producer (a ring of activation windows, two per step, and a ring of weight tiles, one per (slab, tap), shared by
// the two tiles of the pair); warps 1 and 2 = MMA issuers, one per tile of the pair, each with its own accumulator in TMEM
// (a single thread issues a tcgen05.mma only every ~150 cycles, see micro.cu, so one issuer cannot keep the tensor core busy);
// warps 3..10 = two epilogue groups of four warps, one per tile of the pair (TMEM -> registers -> scale, residual add, bf16 ->
// 16 KB staging slabs of 64 columns -> TMA store or row copy-out, with per-tile column sums for the BN that follows).
// The weight-gradient kernel (192 threads) has one producer warp, one issuer warp and four epilogue warps.
// Every wait is bounded: on expiry the kernel records the place in the status word, drains its copies and MMAs, frees its
// TMEM and returns.
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
__device__ __forceinline__ void tma_store_2d(const void* tmap, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tmap), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bar_sync_epi(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }   // the four warps of one epilogue group
__device__ __forceinline__ bool bar_and_epi(int id, bool v) {     // barrier of the four warps of an epilogue group that also ANDs a flag
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %2, 0;\n\tbar.red.and.pred q, %1, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}" : "=r"(r) : "r"(id), "r"((uint32_t)v) : "memory");
    return r != 0;
}
__device__ __forceinline__ void bulk_wait_read(int pending) {     // at most `pending` of this thread's latest bulk stores may still be reading shared memory
    if (pending <= 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    else if (pending == 1) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
    else asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t a) { uint4 v; asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a)); return v; }
__device__ __forceinline__ void sts128(uint32_t a, uint4 v) { asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory"); }
__device__ __forceinline__ uint32_t lds32(uint32_t a) { uint32_t v; asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a)); return v; }

constexpr int TC_THREADS = 224;              // wgrad kernel: producer warp, two MMA warps, four epilogue warps
constexpr int TC_MAX_ISSUERS = 2;            // forward / dgrad kernel: MMA-issuing warps, one per tile of a pair
constexpr int TC_CONV_THREADS = 32 * (1 + TC_MAX_ISSUERS + 8);   // forward / dgrad kernel: producer warp, MMA warps, two groups of four epilogue warps
constexpr int TC_MAX_STAGES = 12;
constexpr int TILE_M = 128;
constexpr int SLAB_BYTES = TILE_M * 128;      // 128 rows x 64 channels of bf16

struct TapRef { int wtap; int shift; };       // weight tap index (r*ksz + s); row shift of the operand inside the window
// One forward / dgrad problem.  The tensor maps come first so that each is 64-byte aligned.
//
// Positions and windows.  The positions of a problem are either the pixels of the output in order ("dense": 1x1 layers) or a
// tall map of Hp x Wp positions per image with `pad` zero rows before each image and `pad` zero columns after each row (3x3
// layers).  A tile is 128 consecutive positions [p0, p0 + 128).  Its operand for one tap group is a window of positions
// [p0 - hb, ...) fetched once per 64-channel slab; tap t of the group reads the window from row (p0 - hb - window start) +
// shift[t] on.  Window position (image, yy, xx) holds activation pixel ((yy - pad) * es + gys, xx * es + gxs) of that
// image, zero outside it: es = 2 with one group per input parity phase makes a stride-2 layer exact work (forward), and four
// problems, one per output phase, do the same for a stride-2 dgrad.
struct TcHot {                // everything the kernel's loops read: each role keeps a copy in shared memory
    const __nv_bfloat16* add; __nv_bfloat16* out;
    float* stat_tiles;        // [tiles_m][2][ncol]: column sums and sums of squares of the stored tile, or nullptr
    int* status;
    int a_flat;               // 1: a window is one box of 128 pixels of the (channel, pixel) map
    int dense;                // 1: position index == output pixel index
    int add_mode;             // 0 none; 2 residual read at the output pixel; 3 residual read from a compact tensor that applies at even (y, x) only
    int ngroups; int gbeg[5]; int gxs[4], gys[4];
    int wtap[9], shift[9];    // per tap: weight tap index (r*ksz + s); row shift of the operand inside the window
    int es, pad;
    int Hp, Wp, n_img;
    int R, box_pos, nbox, hb, a_box_bytes;
    int tiles_m, tiles_n, n_tile, ncol;      // output tile grid; MMA N; channels of the output tensor
    int red, slabs;                          // reduction channels, 64-channel slabs
    int b_mn_major;                          // 0: forward (weights K-major); 1: dgrad (weights MN-major)
    int b_bytes;                             // bytes of one weight tile (one slab, one tap)
    int b_total;                             // bytes of all weight tiles of one column tile, each rounded up to 1 KB
    int out_slabs;                           // 64-column slabs of the output tile
    int total_pos;
    float scale;
    int OH, OW, os, oy, ox;                  // position (image, yy, xx) -> output pixel ((yy - pad) * os + oy, xx * os + ox) of an OH x OW image
};
struct alignas(64) TcProb {
    CUtensorMap map_a;        // activations (forward: a; dgrad: dy): (channel, pixel) or (channel, x, y, image), possibly element-strided
    CUtensorMap map_b;        // weights [K][taps][C] viewed as (C, tap, K)
    CUtensorMap map_out;      // dense problems: the output as (channel, pixel), box 64 x 128
    TcHot h;
};
static_assert(sizeof(TcHot) % 4 == 0, "copied word by word");

struct TcLaunch { int nprob, na, nb, a_stage, b_stage, tmem_cols, acc_stride, nbuf, groups, pg; };
// nbuf: accumulators per tile of a pair (2: the next pair's MMAs run under this pair's epilogues); groups: epilogue groups (two: one
// per tile of a pair; one: it takes both tiles in turn); pg: 16 KB staging buffers (one 64-column slab each) per group
constexpr int TC_MAX_PROBS = 128;             // descriptors per launch (sub-ResNets x output phases)

__device__ __forceinline__ void copy_hot(TcHot* dst, const TcHot* src, int tid, int nthreads) {
    const uint32_t* s4 = reinterpret_cast<const uint32_t*>(src); uint32_t* d4 = reinterpret_cast<uint32_t*>(dst);
    for (int i = tid; i < (int)(sizeof(TcHot) / 4); i += nthreads) d4[i] = __ldg(s4 + i);
}

__global__ void __launch_bounds__(TC_CONV_THREADS, 1) conv_tc_kernel(const TcProb* __restrict__ probs, const TcLaunch L) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[4 * TC_MAX_STAGES + 10];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int pix_s2[2][TILE_M];
    __shared__ float stat_s2[2][4][2][256];
    __shared__ int unit_end_s[TC_MAX_PROBS];                      // running sum of the problems' unit counts (a unit: two row tiles x one column tile)
    __shared__ int tilesm_s[TC_MAX_PROBS], tilesn_s[TC_MAX_PROBS];
    __shared__ TcHot hot_s[3 + TC_MAX_ISSUERS];                   // the current problem of the producer, the two epilogue groups, the MMA issuers
    const uint32_t a_full = smem_u32(&bars[0]), a_empty = smem_u32(&bars[TC_MAX_STAGES]);
    const uint32_t b_full = smem_u32(&bars[2 * TC_MAX_STAGES]), b_empty = smem_u32(&bars[3 * TC_MAX_STAGES]);
    const uint32_t acc_full = smem_u32(&bars[4 * TC_MAX_STAGES]), acc_empty = smem_u32(&bars[4 * TC_MAX_STAGES + 4]);
    const uint32_t drain = smem_u32(&bars[4 * TC_MAX_STAGES + 8]);
    const uint32_t a_ring = smem_u32(smem), b_ring = a_ring + (uint32_t)(L.na * L.a_stage), stg_base = b_ring + (uint32_t)(L.nb * L.b_stage);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) {
            mbar_init(a_full + 8 * s, 1); mbar_init(a_empty + 8 * s, 1); mbar_init(b_full + 8 * s, 1);
            mbar_init(b_empty + 8 * s, TC_MAX_ISSUERS);          // a weight tile serves both tiles of a pair: both issuers release it
        }
        for (int s = 0; s < 4; ++s) { mbar_init(acc_full + 8 * s, 1); mbar_init(acc_empty + 8 * s, 4); }
        for (int s = 0; s < TC_MAX_ISSUERS; ++s) mbar_init(drain + 8 * s, 1);
        abort_s = 0;
        int run = 0;
        for (int i = 0; i < L.nprob; ++i) {
            const TcHot* hp = &probs[i].h;
            run += ((hp->tiles_m + 1) >> 1) * hp->tiles_n; unit_end_s[i] = run;
            tilesm_s[i] = hp->tiles_m; tilesn_s[i] = hp->tiles_n;
        }
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
    // A unit of work is a pair of neighbouring row tiles (2 x 128 positions) times one column tile: the two tiles share every weight
    // tile, which is fetched once, and each has its own MMA-issuing warp and accumulator.  (One thread issues a tcgen05.mma only every
    // ~150 cycles whatever its N (measured), more than the tensor core needs for it: two issuers keep it busy, and each tile's sum
    // is still formed by one thread in a fixed order.)  The units of all problems, column tile innermost, are dealt round-robin: the
    // CTAs that run side by side work on neighbouring tiles, share windows and weight tiles in L2 and read HBM as one moving front.
    // (Contiguous runs per CTA, with the column tile outermost, were measured too: no faster, and slower where the weights stream.)
    const int u_begin = (int)blockIdx.x, u_stop = unit_end_s[L.nprob - 1], u_step = (int)gridDim.x;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t a_cnt = 0, b_cnt = 0; bool ok = true;
            int cur = -1; TcHot& h = hot_s[0];
            int sa = 0, sb_ = 0; uint32_t pha = 0, phb = 0;       // ring positions and phases
            for (int u = u_begin; u < u_stop && ok; u += u_step) {
                int pi = 0; while (u >= unit_end_s[pi]) ++pi;
                if (pi != cur) { copy_hot(&h, &probs[pi].h, 0, 1); cur = pi; }
                const TcProb* pp = probs + pi;
                const int loc = u - (pi ? unit_end_s[pi - 1] : 0);
                const int n_tile = h.n_tile, slabs = h.slabs, ngroups = h.ngroups, a_flat = h.a_flat, nbox = h.nbox,
                          a_box_bytes = h.a_box_bytes, R = h.R, Hp = h.Hp, pad = h.pad, es = h.es, b_bytes = h.b_bytes, mn = h.b_mn_major;
                const int tiles_n = h.tiles_n, tn = loc % tiles_n, tm0 = 2 * (loc / tiles_n), nt = tm0 + 1 < h.tiles_m ? 2 : 1;
                for (int sl = 0; sl < slabs && ok; ++sl) {
                    for (int g = 0; g < ngroups && ok; ++g) {
                        for (int j = 0; j < nt; ++j) {
                            if (!mbar_wait(a_empty + 8 * sa, pha ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 1); ok = false; break; }
                            const int tm = tm0 + j;
                            const uint32_t dst = a_ring + (uint32_t)(sa * L.a_stage);
                            mbar_expect_tx(a_full + 8 * sa, (uint32_t)(nbox * a_box_bytes));
                            if (a_flat) tma_load_2d(dst, &pp->map_a, a_full + 8 * sa, sl * 64, tm * TILE_M);
                            else {
                                const int gx = h.gxs[g], gy = h.gys[g], bx0 = floor_div(tm * TILE_M - h.hb, h.box_pos);
                                for (int i = 0; i < nbox; ++i) {
                                    const int trow = (bx0 + i) * R, img = floor_div(trow, Hp), yy0 = trow - img * Hp;
                                    tma_load_4d(dst + (uint32_t)(i * a_box_bytes), &pp->map_a, a_full + 8 * sa, sl * 64, gx, (yy0 - pad) * es + gy, img);
                                }
                            }
                            ++a_cnt; if (++sa == L.na) { sa = 0; pha ^= 1u; }
                        }
                        if (!ok) break;
                        const int t_end = h.gbeg[g + 1];
                        for (int tap = h.gbeg[g]; tap < t_end; ++tap) {
                            if (!mbar_wait(b_empty + 8 * sb_, phb ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 2); ok = false; break; }
                            const uint32_t dst = b_ring + (uint32_t)(sb_ * L.b_stage);
                            const int wtap = h.wtap[tap];
                            mbar_expect_tx(b_full + 8 * sb_, (uint32_t)b_bytes);
                            if (!mn) tma_load_3d(dst, &pp->map_b, b_full + 8 * sb_, sl * 64, wtap, tn * n_tile);
                            else for (int c = 0; c * 64 < n_tile; ++c)
                                tma_load_3d(dst + (uint32_t)(c * 8192), &pp->map_b, b_full + 8 * sb_, tn * n_tile + c * 64, wtap, sl * 64);
                            ++b_cnt; if (++sb_ == L.nb) { sb_ = 0; phb ^= 1u; }
                        }
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
    } else if (warp <= TC_MAX_ISSUERS) {
        // ---------------------------------------------------------------- MMA issuers: warp 1 + j runs the reduction of tile j of every
        // pair into its own accumulator.  Windows are per tile (the pair's two windows sit in consecutive ring stages); a weight stage
        // is read by both issuers and released by both (an issuer whose pair has no second tile only passes the weight stages on).
        const int me = warp - 1;
        if (lane == 0) {
            uint32_t a_cnt = 0, cnt = 0; bool ok = true;
            int cur = -1; TcHot& h = hot_s[3 + me];
            int sb = 0; uint32_t phb = 0;
            // the constant part of a 128-byte-swizzle descriptor: stride between 8-row groups 1024 bytes, version, swizzle mode
            const uint64_t desc_k = desc_sw128(0, 16, 1024), desc_mn = desc_sw128(0, 8192, 1024);
            for (int u = u_begin; u < u_stop && ok; u += u_step) {
                int pi = 0; while (u >= unit_end_s[pi]) ++pi;
                if (pi != cur) { copy_hot(&h, &probs[pi].h, 0, 1); cur = pi; }
                const int loc = u - (pi ? unit_end_s[pi - 1] : 0);
                const int slabs = h.slabs, ngroups = h.ngroups, red = h.red, mn = h.b_mn_major;
                const int tm0 = 2 * (loc / h.tiles_n), nt = tm0 + 1 < h.tiles_m ? 2 : 1, tm = tm0 + me;
                const bool has = me < nt;
                const int bx0 = h.a_flat ? 0 : floor_div(tm * TILE_M - h.hb, h.box_pos);
                const int a_off = h.a_flat ? 0 : tm * TILE_M - h.hb - bx0 * h.box_pos;
                const uint32_t buf = (cnt % (uint32_t)L.nbuf) * 2u + (uint32_t)me, aph = (cnt / (uint32_t)L.nbuf) & 1u;
                if (has) {
                    ++cnt;
                    if (!mbar_wait(acc_empty + 8 * buf, aph ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 3); ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                }
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)L.acc_stride;
                // instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B K-major or MN-major, N, M = 128
                const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)mn << 16) |
                                       ((uint32_t)(h.n_tile >> 3) << 17) | ((128u >> 4) << 24);
                const uint64_t b_const = mn ? desc_mn : desc_k;
                const uint32_t b_step = mn ? 128u : 2u;           // one K = 16 step: 16 rows of 128 bytes (MN-major) or 32 bytes along the row (K-major), in 16-byte units
                uint32_t acc = 0;
                for (int sl = 0; sl < slabs && ok; ++sl) {
                    const int ksteps = (min(64, red - sl * 64) + 15) >> 4;
                    for (int g = 0; g < ngroups && ok; ++g) {
                        const uint32_t ai = a_cnt + (uint32_t)me; a_cnt += (uint32_t)nt;
                        const uint32_t sa = ai % (uint32_t)L.na, pha = (ai / (uint32_t)L.na) & 1u;
                        if (has) {
                            if (!mbar_wait(a_full + 8 * sa, pha, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 4); ok = false; break; }
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        }
                        const uint32_t a_rows16 = ((a_ring + sa * (uint32_t)L.a_stage) >> 4) + (uint32_t)a_off * 8u;   // start address in 16-byte units
                        const int t_end = h.gbeg[g + 1];
                        for (int tap = h.gbeg[g]; tap < t_end; ++tap) {
                            if (!mbar_wait(b_full + 8 * sb, phb, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 5); ok = false; break; }
                            if (has) {
                                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                                const uint32_t a16 = a_rows16 + (uint32_t)h.shift[tap] * 8u;
                                const uint32_t b16 = (b_ring + (uint32_t)(sb * L.b_stage)) >> 4;
                                for (int k16 = 0; k16 < ksteps; ++k16) {
                                    umma_bf16(d_tmem, desc_k | (uint64_t)((a16 + 2u * (uint32_t)k16) & 0x3FFFu), b_const | (uint64_t)((b16 + b_step * (uint32_t)k16) & 0x3FFFu), idesc, acc);
                                    acc = 1;
                                }
                                umma_commit(b_empty + 8 * sb);   // this issuer's share of the release: once its MMAs have read the weight tile
                            } else mbar_arrive(b_empty + 8 * sb);
                            if (++sb == L.nb) { sb = 0; phb ^= 1u; }
                        }
                        if (has && ok) umma_commit(a_empty + 8 * sa);
                    }
                }
                if (has && ok) umma_commit(acc_full + 8 * buf);  // accumulator complete
            }
            if (!ok) {
                // gave up: the MMAs already issued must have finished before the CTA frees its tensor memory
                umma_commit(drain + 8 * me);
                for (int i = 0; i < 65536 && !mbar_try(drain + 8 * me, 0u); ++i) __nanosleep(64);
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue: two groups of 4 warps (one TMEM lane quadrant each);
        // group g takes tile g of every pair, so two epilogues run side by side (a single group takes both tiles in turn)
        const int grp = (warp - 1 - TC_MAX_ISSUERS) >> 2, bid = 1 + grp;
        const int quad = warp & 3;
        const int m = quad * 32 + lane;                          // row of the tile = TMEM lane
        const int et = threadIdx.x - 32 * (1 + TC_MAX_ISSUERS) - grp * 128;   // 0..127 among the group's threads
        const bool leader = et == 0;
        int* const pix_s = pix_s2[grp];
        float (*const stat_s)[2][256] = stat_s2[grp];
        bool ok = true;
        int cur = -1; const TcHot& h = hot_s[1 + grp];
        uint32_t sc = 0, cnt[2] = {0u, 0u};                      // 64-column slabs this group has staged; tiles taken of each half of the pairs
        for (int u = u_begin; grp < L.groups && u < u_stop && ok; u += u_step) {
          int pi = 0; while (u >= unit_end_s[pi]) ++pi;
          const TcProb* pp = probs + pi;
          const int loc = u - (pi ? unit_end_s[pi - 1] : 0);
          const int tn = loc % tilesn_s[pi], tm0 = 2 * (loc / tilesn_s[pi]), nt = tm0 + 1 < tilesm_s[pi] ? 2 : 1;
          for (int hf = L.groups == 2 ? grp : 0; hf < nt && ok; hf += L.groups == 2 ? 2 : 1) {
            const int tm = tm0 + hf;
            const uint32_t buf = (cnt[hf] % (uint32_t)L.nbuf) * 2u + (uint32_t)hf, aph = (cnt[hf] / (uint32_t)L.nbuf) & 1u;
            ++cnt[hf];
            // every warp must have finished its share of the last tile's copy-out (it reads the pixel table)
            bar_sync_epi(bid);
            if (pi != cur) { copy_hot(&hot_s[1 + grp], &probs[pi].h, et, 128); cur = pi; bar_sync_epi(bid); }
            const int n_tile = h.n_tile, ncol = h.ncol, add_mode = h.add_mode, dense = h.dense;
            const float scale = h.scale;
            const __nv_bfloat16* addp = h.add; __nv_bfloat16* outp = h.out; float* stat_tiles = h.stat_tiles;
            // position -> output pixel (and the residual's pixel)
            const int pos = tm * TILE_M + m;
            bool valid = pos < h.total_pos;
            long long pix = pos, addpix = -1;
            if (valid && (!dense || add_mode == 3)) {
                const int Wp = h.Wp, Hp = h.Hp, pad = h.pad, os = h.os, OH = h.OH, OW = h.OW;
                const int trow = pos / Wp, xx = pos - trow * Wp, img = trow / Hp, yy = trow - img * Hp;
                const int y = (yy - pad) * os + h.oy, x = xx * os + h.ox;
                valid = yy >= pad && xx < Wp - pad && y < OH && x < OW;
                pix = ((long long)img * OH + y) * OW + x;
                if (add_mode == 3 && !((y | x) & 1)) addpix = ((long long)img * ((OH + 1) >> 1) + (y >> 1)) * ((OW + 1) >> 1) + (x >> 1);
            }
            if (add_mode == 2) addpix = pix;
            if (!dense) pix_s[m] = valid ? (int)pix : -1;
            const int col0 = tn * n_tile;
            const bool gadd = add_mode >= 2 && valid && addpix >= 0;
            // the residual of a 32-column step is fetched one step ahead of its use (the first one ahead of the accumulator)
            const __nv_bfloat16* addrow = addp + (gadd ? addpix : 0) * ncol + col0;
            uint4 ga[4], gn[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) gn[g] = (gadd && g * 8 < n_tile && col0 + g * 8 < ncol) ? __ldg(reinterpret_cast<const uint4*>(addrow + g * 8)) : make_uint4(0u, 0u, 0u, 0u);
            if (add_mode == 2 && dense) {
                // the residual rows of the group's next tile are asked into L2 now, a whole tile ahead of their use
                int u2 = u, hf2 = hf + (L.groups == 2 ? 2 : 1);
                if (hf2 >= nt) { u2 = u + u_step; hf2 = L.groups == 2 ? grp : 0; }
                if (u2 < unit_end_s[pi]) {                       // same problem (else the next tile's own first loads have to do)
                    const int loc2 = u2 - (pi ? unit_end_s[pi - 1] : 0);
                    const int tn2 = loc2 % tilesn_s[pi], tm2 = 2 * (loc2 / tilesn_s[pi]) + hf2;
                    const long long pos2 = (long long)tm2 * TILE_M + m;
                    if (tm2 < tilesm_s[pi] && pos2 < h.total_pos) {
                        const __nv_bfloat16* r2 = addp + pos2 * ncol + tn2 * n_tile;
                        for (int c = 0; c < n_tile && tn2 * n_tile + c < ncol; c += 64)
                            asm volatile("prefetch.global.L2 [%0];" ::"l"(r2 + c));
                    }
                }
            }
            ok = mbar_wait(acc_full + 8 * buf, aph, &abort_s);
            ok = bar_and_epi(bid, ok);                           // one decision for the four warps: they share the barriers below
            if (!ok) { atomicExch(&abort_s, 1); atomicExch(h.status, 6); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t t_row = tmem_base + buf * (uint32_t)L.acc_stride + ((uint32_t)(quad * 32) << 16);
            // The tile leaves in slabs of 64 columns: a slab is rounded and (with the residual added) written to a 16 KB staging
            // buffer in the 128-byte-swizzle layout, then stored by TMA (dense problems) or copied out row by row, while the next
            // slab is staged in the group's other buffer.
            for (int c0 = 0; c0 < n_tile; c0 += 32) {
                const int slab = c0 >> 6;
                const bool slab_begin = !(c0 & 32), slab_end = (c0 & 32) || c0 + 32 >= n_tile, last = c0 + 32 >= n_tile;
                const uint32_t stg = stg_base + ((uint32_t)(grp * L.pg) + sc % (uint32_t)L.pg) * SLAB_BYTES;
                if (slab_begin) {
                    if (leader) bulk_wait_read(L.pg - 1);        // the bulk store issued from this buffer has read it
                    bar_sync_epi(bid);                           // ... and every warp is done with what it last held
                }
                uint32_t v[32];
                tmem_ld32(t_row + (uint32_t)c0, v);
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    ga[g] = gn[g];
                    const int c = c0 + 32 + g * 8;
                    gn[g] = (gadd && c < n_tile && col0 + c < ncol) ? __ldg(reinterpret_cast<const uint4*>(addrow + c)) : make_uint4(0u, 0u, 0u, 0u);
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (last) {
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_empty + 8 * buf); // this warp has read its quadrant of the accumulator
                }
                const uint32_t s_row = stg + (uint32_t)m * 128u;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int c = c0 + g * 8;
                    if (c < n_tile) {
                        const uint32_t sa = s_row + ((uint32_t)(((c >> 3) & 7) ^ (m & 7)) << 4);
                        float f[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) f[k] = valid ? __uint_as_float(v[g * 8 + k]) * scale : 0.f;
                        if (gadd) {
                            const uint32_t aw[4] = {ga[g].x, ga[g].y, ga[g].z, ga[g].w};
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                f[2 * k] += __uint_as_float(aw[k] << 16);
                                f[2 * k + 1] += __uint_as_float(aw[k] & 0xFFFF0000u);
                            }
                        }
                        uint32_t w[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            __nv_bfloat162 hh = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
                            w[k] = *reinterpret_cast<uint32_t*>(&hh);
                        }
                        sts128(sa, make_uint4(w[0], w[1], w[2], w[3]));
                    }
                }
                if (!slab_end) continue;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the bulk store reads what this thread wrote
                bar_sync_epi(bid);                               // the slab is complete
                if (dense && leader) {
                    tma_store_2d(&pp->map_out, stg, col0 + slab * 64, tm * TILE_M);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                if (stat_tiles) {
                    // column sums of the stored (rounded) values: every warp over its own 32 rows, lane = two neighbouring columns;
                    // the four warps' sums are added in a fixed order once the tile's last slab is through
                    float s0 = 0.f, s1 = 0.f, q0 = 0.f, q1 = 0.f;
#pragma unroll 8
                    for (int r = 0; r < 32; ++r) {
                        const int row = quad * 32 + r;
                        const uint32_t uu = lds32(stg + (uint32_t)row * 128u + ((uint32_t)((lane >> 2) ^ (row & 7)) << 4) + ((uint32_t)(lane & 3) << 2));
                        const float lo = __uint_as_float(uu << 16), hi = __uint_as_float(uu & 0xFFFF0000u);
                        s0 += lo; q0 += lo * lo; s1 += hi; q1 += hi * hi;
                    }
                    stat_s[quad][0][slab * 64 + 2 * lane] = s0; stat_s[quad][0][slab * 64 + 2 * lane + 1] = s1;
                    stat_s[quad][1][slab * 64 + 2 * lane] = q0; stat_s[quad][1][slab * 64 + 2 * lane + 1] = q1;
                }
                if (!dense) {
                    // copy-out of a tall slab: 16-byte chunks, eight consecutive lanes per 128-byte run of one output pixel
                    for (int idx = et; idx < TILE_M * 8; idx += 128) {
                        const int ch = idx & 7, row = idx >> 3;
                        const int c = slab * 64 + ch * 8, px = pix_s[row];
                        if (px >= 0 && c < n_tile && col0 + c < ncol)
                            *reinterpret_cast<uint4*>(outp + (long long)px * ncol + col0 + c) =
                                lds128(stg + (uint32_t)row * 128u + ((uint32_t)(ch ^ (row & 7)) << 4));
                    }
                }
                ++sc;
            }
            if (stat_tiles) {
                bar_sync_epi(bid);
                for (int c = et; c < n_tile; c += 128) {
                    if (col0 + c < ncol) {
                        const float su = ((stat_s[0][0][c] + stat_s[1][0][c]) + stat_s[2][0][c]) + stat_s[3][0][c];
                        const float sq = ((stat_s[0][1][c] + stat_s[1][1][c]) + stat_s[2][1][c]) + stat_s[3][1][c];
                        stat_tiles[((long long)tm * 2 + 0) * ncol + col0 + c] = su;
                        stat_tiles[((long long)tm * 2 + 1) * ncol + col0 + c] = sq;
                    }
                }
            }
          }
        }
        if (leader) bulk_wait_read(0);                           // shared memory stays until the last bulk stores have read it
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
// positions of the forward problem (pixels in order, or the tall zero-padded map, where dy reads as zero at the padding
// positions and adds nothing), 128 per pipeline stage: D[cout (128 lanes), cin] per tap, A = dy^T and B = shifted a,
// both MN-major straight from their 128-byte rows.  A CTA accumulates a range of position chunks for one group of taps
// (taps that read the same window: up to three taps of a stride-1 layer, the taps of one input parity phase of a stride-2
// layer) and writes an fp32 partial, or, alone on its tile, the result; a second kernel adds the partials in a fixed order.
struct alignas(64) TcWgradProb {
    CUtensorMap map_dy;       // (channel k, pixel) or (channel k, x, y, image)
    CUtensorMap map_a;        // likewise for a, possibly element-strided
    float* partial;           // [splits][taps][cout][cin]
    float* out;               // [cout][taps][cin]
    int* status;
    int dy_flat, a_flat, taps;
    int es, pad, Hp, Wp, n_img;
    int R, box_pos, nbox_dy, nbox_a, hb, dy_box_bytes, a_box_bytes;
    int chunks;                                   // position chunks of 128 in total
    int cout, cin, m_tiles, n_tile, n_tiles, a_slabs;
    int tap_groups; int gbeg[10]; int gxs[9], gys[9];
    TapRef tap[9];                                // wtap = index of the tap in dw; shift = row shift inside the a window
    int splits, chunks_per_split;
    int dy_slab_bytes, a_slab_bytes;              // one 64-channel slab of a stage
    int stage_bytes, stages, tmem_cols;
};

__global__ void __launch_bounds__(TC_THREADS, 1) conv_wgrad_tc_kernel(const TcWgradProb* __restrict__ probs) {
    const TcWgradProb& p = probs[blockIdx.y];
    const int ctas = p.m_tiles * p.n_tiles * p.tap_groups * p.splits;
    if ((int)blockIdx.x >= ctas) return;
    // everything the loops read, in registers (the descriptor lives in global memory)
    const int splits = p.splits, tap_groups = p.tap_groups, n_tiles = p.n_tiles, chunks = p.chunks, chunks_per_split = p.chunks_per_split;
    const int stages = p.stages, stage_bytes = p.stage_bytes, dy_slab_bytes = p.dy_slab_bytes, a_slab_bytes = p.a_slab_bytes, a_slabs = p.a_slabs;
    const int n_tile = p.n_tile, dy_flat = p.dy_flat, a_flat = p.a_flat, box_pos = p.box_pos, hb = p.hb, R = p.R, Hp = p.Hp, pad = p.pad, es = p.es;
    const int nbox_dy = p.nbox_dy, nbox_a = p.nbox_a, dy_box_bytes = p.dy_box_bytes, a_box_bytes = p.a_box_bytes, tmem_cols = p.tmem_cols;
    int id = blockIdx.x;
    const int split = id % splits; id /= splits;
    const int tg = id % tap_groups; id /= tap_groups;
    const int tn = id % n_tiles; const int tm = id / n_tiles;
    const int c_begin = split * chunks_per_split;
    const int c_end = min(c_begin + chunks_per_split, chunks);
    const int tap0 = p.gbeg[tg], ntap = p.gbeg[tg + 1] - tap0;
    const int gx = p.gxs[tg], gy = p.gys[tg];
    const int nc = c_end - c_begin;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[2 * TC_MAX_STAGES + 3];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int shift8_s[4], wtap_s[4];                       // the group's taps: row shift in 16-byte units, index in dw
    const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[TC_MAX_STAGES]), bar_acc = smem_u32(&bars[2 * TC_MAX_STAGES]);
    const uint32_t bar_drain = smem_u32(&bars[2 * TC_MAX_STAGES + 1]);
    const uint32_t ring = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 2); }   // both issuers release a stage
        mbar_init(bar_acc, 2); mbar_init(bar_drain, 1); mbar_init(bar_drain + 8, 1);
        abort_s = 0;
        for (int i = 0; i < ntap; ++i) { shift8_s[i] = p.tap[tap0 + i].shift * 8; wtap_s[i] = p.tap[tap0 + i].wtap; }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_s;

    if (warp == 0) {
        if (lane == 0) {
            int i = 0; bool ok = true; int s = 0; uint32_t ph = 0;
            const uint32_t tx = (uint32_t)(2 * nbox_dy * dy_box_bytes + a_slabs * nbox_a * a_box_bytes);
            for (; i < nc; ++i) {
                if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 11); ok = false; break; }
                const int pos0 = (c_begin + i) * TILE_M;
                const uint32_t dy_dst = ring + (uint32_t)(s * stage_bytes), a_dst = dy_dst + 2u * (uint32_t)dy_slab_bytes;
                mbar_expect_tx(bar_full + 8 * s, tx);
                if (dy_flat) {
                    for (int j = 0; j < 2; ++j) tma_load_2d(dy_dst + (uint32_t)(j * dy_slab_bytes), &p.map_dy, bar_full + 8 * s, tm * 128 + j * 64, pos0);
                } else {
                    const int bd0 = pos0 / box_pos;
                    for (int b = 0; b < nbox_dy; ++b) {
                        const int trow = (bd0 + b) * R, img = trow / Hp, yy0 = trow - img * Hp;
                        for (int j = 0; j < 2; ++j)
                            tma_load_4d(dy_dst + (uint32_t)(j * dy_slab_bytes + b * dy_box_bytes), &p.map_dy, bar_full + 8 * s, tm * 128 + j * 64, 0, yy0 - pad, img);
                    }
                }
                if (a_flat) {
                    for (int j = 0; j < a_slabs; ++j) tma_load_2d(a_dst + (uint32_t)(j * a_slab_bytes), &p.map_a, bar_full + 8 * s, tn * n_tile + j * 64, pos0);
                } else {
                    const int ba0 = floor_div(pos0 - hb, box_pos);
                    for (int b = 0; b < nbox_a; ++b) {
                        const int trow = (ba0 + b) * R, img = floor_div(trow, Hp), yy0 = trow - img * Hp;
                        for (int j = 0; j < a_slabs; ++j)
                            tma_load_4d(a_dst + (uint32_t)(j * a_slab_bytes + b * a_box_bytes), &p.map_a, bar_full + 8 * s, tn * n_tile + j * 64,
                                        gx, (yy0 - pad) * es + gy, img);
                    }
                }
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
            if (!ok)
                for (int c = max(0, i - stages); c < i; ++c)
                    for (int w = 0; w < 4096 && !mbar_try(bar_full + 8 * (c % stages), (uint32_t)(c / stages) & 1u); ++w) __nanosleep(64);
        }
    } else if (warp <= 2) {
        // Two issuing warps (one thread issues a tcgen05.mma only every ~150 cycles, more than the tensor core needs for it).  The
        // group's taps are split between them; with an odd number of taps the last tap's 128 positions are split instead, each
        // half into an accumulator of its own (the epilogue adds the two, first half first).  So every accumulator is written
        // by one thread, in a fixed order.
        if (lane == 0) {
            const int me = warp - 1, odd = ntap & 1, whole = (ntap - odd) >> 1;
            int it_tap[3], it_acc[3], it_k0[3], it_k1[3], nit = 0;
            for (int q = 0; q < whole; ++q) { it_tap[nit] = me * whole + q; it_acc[nit] = me * whole + q; it_k0[nit] = 0; it_k1[nit] = 8; ++nit; }
            if (odd) { it_tap[nit] = ntap - 1; it_acc[nit] = ntap - 1 + me; it_k0[nit] = me * 4; it_k1[nit] = me * 4 + 4; ++nit; }
            // fp32 accumulate, bf16 x bf16, A and B MN-major, N = n_tile, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(n_tile >> 3) << 17) | ((128u >> 4) << 24);
            const uint64_t dy_const = desc_sw128(0, (uint32_t)dy_slab_bytes, 1024), a_const = desc_sw128(0, (uint32_t)a_slab_bytes, 1024);
            bool ok = true; int s = 0; uint32_t ph = 0;
            for (int i = 0; i < nc && ok; ++i) {
                if (!mbar_wait(bar_full + 8 * s, ph, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(p.status, 12); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const int pos0 = (c_begin + i) * TILE_M;
                const int dy_off = dy_flat ? 0 : pos0 - (pos0 / box_pos) * box_pos;
                const int a_off = a_flat ? 0 : pos0 - hb - floor_div(pos0 - hb, box_pos) * box_pos;
                const uint32_t dy16 = ((ring + (uint32_t)(s * stage_bytes)) >> 4) + (uint32_t)dy_off * 8u;       // start addresses in 16-byte units
                const uint32_t a16 = ((ring + (uint32_t)(s * stage_bytes) + 2u * (uint32_t)dy_slab_bytes) >> 4) + (uint32_t)a_off * 8u;
                for (int q = 0; q < nit; ++q) {
                    const uint32_t at16 = a16 + (uint32_t)shift8_s[it_tap[q]];
                    const uint32_t d_t = tmem_d + (uint32_t)(it_acc[q] * n_tile);
                    const int k0 = it_k0[q], k1 = it_k1[q];
                    for (int k16 = k0; k16 < k1; ++k16)        // 16 positions = 16 rows of 128 bytes per step
                        umma_bf16(d_t, dy_const | (uint64_t)((dy16 + 128u * (uint32_t)k16) & 0x3FFFu), a_const | (uint64_t)((at16 + 128u * (uint32_t)k16) & 0x3FFFu), idesc, (i || k16 != k0) ? 1u : 0u);
                }
                umma_commit(bar_empty + 8 * s);
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(bar_acc);
            else {
                // gave up: the MMAs already issued must have finished before the CTA frees its tensor memory
                umma_commit(bar_drain + 8 * me);
                for (int w = 0; w < 65536 && !mbar_try(bar_drain + 8 * me, 0u); ++w) __nanosleep(64);
            }
        }
    } else {
        const int quad = warp & 3, m = quad * 32 + lane;
        const int cout = p.cout, cin = p.cin, taps = p.taps;
        float* const partial = p.partial; float* const outp = p.out;
        bool ok = nc > 0 ? mbar_wait(bar_acc, 0, &abort_s) : true;
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { atomicExch(&abort_s, 1); atomicExch(p.status, 13); }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int k = tm * 128 + m;
        if (ok && quad * 32 < cout - tm * 128) {              // warp-uniform: this lane quadrant holds real output channels
            for (int tt = 0; tt < ntap; ++tt) {
                const int wt = wtap_s[tt];
                float* dst = splits > 1 ? partial + (((long long)split * taps + wt) * cout + k) * cin + tn * n_tile
                                        : outp + ((long long)k * taps + wt) * cin + tn * n_tile;
                for (int c0 = 0; c0 < n_tile; c0 += 32) {
                    uint32_t v[32];
                    if (nc > 0) {
                        tmem_ld32(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(tt * n_tile + c0), v);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        if ((ntap & 1) && tt == ntap - 1) {      // the tap whose positions were split: first half + second half
                            uint32_t v2[32];
                            tmem_ld32(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ntap * n_tile + c0), v2);
                            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(v2[j]));
                        }
                    } else { for (int j = 0; j < 32; ++j) v[j] = 0u; }
                    if (k < cout) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (c0 + j < n_tile && tn * n_tile + c0 + j < cin)
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(tmem_cols) : "memory");
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

// ------------------------------------------------------------------------------------------------ BN statistics from the tiles' sums
// The forward kernel leaves, per 128-position tile, the column sums and sums of squares of the values it stored.  One warp
// per channel adds them in a fixed order in double and turns them into mean, 1/sqrt(var + eps) and the running statistics.
__global__ void __launch_bounds__(256) bn_finalize_tiles_kernel(const BnProb* __restrict__ probs) {
    const BnProb& p = probs[blockIdx.y];
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (c >= p.C) return;
    const float* tiles = reinterpret_cast<const float*>(p.partial);
    double a0 = 0.0, a1 = 0.0;
    for (int k = lane; k < p.chunks; k += 32) { a0 += (double)tiles[((long long)k * 2 + 0) * p.C + c]; a1 += (double)tiles[((long long)k * 2 + 1) * p.C + c]; }
    for (int d = 16; d; d >>= 1) { a0 += __shfl_xor_sync(0xffffffffu, a0, d); a1 += __shfl_xor_sync(0xffffffffu, a1, d); }
    if (lane != 0) return;
    const double m = (double)p.m, mean = a0 / m;
    double var = a1 / m - mean * mean; if (var < 0.0) var = 0.0;
    p.stat[c] = (float)mean;
    p.stat[p.C + c] = (float)(1.0 / sqrt(var + (double)p.eps));
    if (p.run_mean) {
        const double unb = p.m > 1 ? var * m / (m - 1.0) : var, mo = (double)p.momentum;
        p.run_mean[c] = (float)((1.0 - mo) * (double)p.run_mean[c] + mo * mean);
        p.run_var[c] = (float)((1.0 - mo) * (double)p.run_var[c] + mo * unb);
    }
}
void launch_bn_finalize_tiles(const BnProb* d, int nprob, int max_c, cudaStream_t s) {
    bn_finalize_tiles_kernel<<<dim3((max_c + 7) / 8, nprob), 256, 0, s>>>(d);
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

// bf16 tensor map of `rank` dimensions (innermost first), 128-byte swizzle, zero fill out of bounds; estr = traversal strides
static bool encode_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box,
                       const uint32_t* estr = nullptr) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t d[5]; cuuint64_t st[4]; cuuint32_t b[5]; cuuint32_t es[5];
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = estr ? estr[i] : 1; if (i + 1 < rank) st[i] = strides_bytes[i]; }
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// [pixels][chan] as (channel, pixel), box 64 x 128
static bool encode_flat(CUtensorMap* m, const void* base, int chan, long long pixels) {
    const uint64_t dims[2] = {(uint64_t)chan, (uint64_t)pixels}; const uint64_t st[1] = {(uint64_t)chan * 2}; const uint32_t box[2] = {64, 128};
    return encode_map(m, base, 2, dims, st, box);
}
// [n_img][H][W][chan] as (channel, x, y, image): a box is box_h rows of Wp window positions of box_n images, every es-th pixel in x and y
static bool encode_tall(CUtensorMap* m, const void* base, int chan, int n_img, int H, int W, int Wp, int box_h, int box_n, int es) {
    const uint64_t dims[4] = {(uint64_t)chan, (uint64_t)W, (uint64_t)H, (uint64_t)n_img};
    const uint64_t st[3] = {(uint64_t)chan * 2, (uint64_t)chan * 2 * W, (uint64_t)chan * 2 * W * H};
    const uint32_t box[4] = {64, (uint32_t)(Wp * es), (uint32_t)(box_h * es), (uint32_t)box_n};
    const uint32_t estr[4] = {1, (uint32_t)es, (uint32_t)es, 1};
    return encode_map(m, base, 4, dims, st, box, estr);
}

// The tall map of a grid of Hg x Wg positions per image: Wp = Wg + pad positions per row, Hp rows per image (Hg + pad, rounded up
// to a multiple of the rows of a box: the extra rows read as zero like the padding).  A box is R consecutive tall rows: part of
// one image (R divides Hp), or box_n whole images.  Larger boxes mean fewer TMA issues per window but more rows fetched around it;
// the choice: at most 96 positions per box, at most 6.5 % of extra rows, then the largest box.
struct Tall { int Hp, Wp, R, box_pos, box_bytes, box_h, box_n; };
static bool tall_of(int Hg, int Wg, int pad, int es, Tall& t, int max_box = 96) {
    t.Wp = Wg + pad;
    const int H0 = Hg + pad;
    if (t.Wp * es > 256) return false;
    int best_r = 1, best_hp = H0;
    for (int r = 1; r <= H0; ++r) {
        const int hp = (H0 + r - 1) / r * r;
        if ((r > 1 && r * t.Wp > max_box) || r * t.Wp > 96 || r * es > 256 || (hp - H0) * 200 > 13 * H0 || (pad == 0 && hp != H0)) continue;   // pad = 0: positions are the pixels in order, no extra rows
        if (r * t.Wp > best_r * t.Wp) { best_r = r; best_hp = hp; }
    }
    t.Hp = best_hp; t.R = best_r; t.box_h = best_r; t.box_n = 1;
    if (best_r == best_hp) {                      // whole images: several per box when they are small
        int ni = max_box / (t.Hp * t.Wp); if (ni < 1) ni = 1; if (ni > 8) ni = 8;
        t.box_n = ni; t.R = t.Hp * ni;
    }
    t.box_pos = t.R * t.Wp; t.box_bytes = t.box_pos * 128;
    return true;
}
static int boxes_for(int span, int box_pos) { return (span + 2 * (box_pos - 1)) / box_pos; }   // boxes that cover `span` positions from any start

// The taps of output phase (u, v) of a stride-2 3x3 dgrad (u, v = parity of the input row and column), or of input phase (u, v)
// of a stride-2 3x3 forward / wgrad: tap (r, s) belongs to the phase with (r - 1) = u, (s - 1) = v modulo 2.
static int phase_taps(int u, int v, int rs[4][2]) {
    int n = 0;
    for (int r = 0; r < 3; ++r) for (int s = 0; s < 3; ++s)
        if ((((r - 1) % 2) + 2) % 2 == u && (((s - 1) % 2) + 2) % 2 == v) { rs[n][0] = r; rs[n][1] = s; ++n; }
    return n;
}

static bool tc_shape_ok(const ConvProb& p) {
    if ((p.ksz != 1 && p.ksz != 3) || p.stride < 1 || p.stride > 2) return false;
    if (p.C % 8 || p.K % 8) return false;
    if ((long long)p.N * (p.H + 1) * (p.W + 1) > (1ll << 30)) return false;
    return true;
}

// Number of TcProb descriptors a forward / dgrad problem needs (0: not supported): one, or one per output phase of a stride-2 3x3 dgrad.
int conv_tc_count(const ConvProb& p, int mode) {
    if (mode == CONV_WGRAD || !encode_fn() || !tc_shape_ok(p)) return 0;
    if (((uintptr_t)p.act | (uintptr_t)p.wgt | (uintptr_t)p.out | (uintptr_t)p.add) & 15) return 0;
    Tall t;
    if (p.ksz == 3 && !tall_of(p.stride == 2 ? p.P : p.H, p.stride == 2 ? p.Q : p.W, 1, mode == CONV_FWD ? p.stride : 1, t)) return 0;
    if (p.ksz == 1 && p.stride == 2 && mode == CONV_FWD && !tall_of(p.P, p.Q, 0, 2, t)) return 0;
    return (mode == CONV_DGRAD && p.ksz == 3 && p.stride == 2) ? 4 : 1;
}
bool conv_tc_supported(const ConvProb& p, int mode) { return conv_tc_count(p, mode) > 0; }
// 128-position tiles of a forward problem (the rows of ConvProb::stat_tiles)
int conv_tc_stat_tiles(const ConvProb& p) {
    long long pos = (long long)p.N * p.P * p.Q;
    if (p.ksz == 1 && p.stride == 2) { Tall g; tall_of(p.P, p.Q, 0, 2, g); pos = (long long)p.N * g.Hp * g.Wp; }
    if (p.ksz != 1) { Tall g; tall_of(p.P, p.Q, 1, p.stride, g); pos = (long long)p.N * g.Hp * g.Wp; }
    return (int)((pos + TILE_M - 1) / TILE_M);
}

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

// Fills conv_tc_count() host-side TcProbs for this problem.  Returns the number written (0: not supported or encoding failed).
int conv_tc_fill(const ConvProb& p, int mode, void* host_tc) {
    const int count = conv_tc_count(p, mode);
    if (!count) return 0;
    const int taps = p.ksz * p.ksz;
    const int chan_a = mode == CONV_FWD ? p.C : p.K, ncol = mode == CONV_FWD ? p.K : p.C;
    for (int ph = 0; ph < count; ++ph) {
        TcProb tp; memset(&tp, 0, sizeof(tp)); TcHot& t = tp.h;
        t.add = (const __nv_bfloat16*)p.add; t.out = (__nv_bfloat16*)p.out; t.status = conv_tc_status_word();
        t.stat_tiles = mode == CONV_FWD ? p.stat_tiles : nullptr;
        t.n_img = p.N; t.ncol = ncol; t.red = chan_a; t.slabs = (chan_a + 63) / 64; t.scale = p.scale;
        t.b_mn_major = mode == CONV_DGRAD ? 1 : 0;
        t.es = 1; t.pad = 0; t.os = 1; t.oy = 0; t.ox = 0; t.ngroups = 1; t.gbeg[0] = 0;
        const void* act = p.act;
        long long out_pixels = 0;
        if (p.ksz == 1 && (p.stride == 1 || mode == CONV_DGRAD)) {
            // plain GEMM over the pixels of the operand: forward at stride 1, dgrad at either stride (stride 2: over the P x Q pixels of dy)
            const int Hg = mode == CONV_DGRAD ? p.P : p.H, Wg = mode == CONV_DGRAD ? p.Q : p.W;
            t.a_flat = 1; t.Hp = Hg; t.Wp = Wg; t.R = 0; t.box_pos = TILE_M; t.nbox = 1; t.hb = 0; t.a_box_bytes = SLAB_BYTES;
            t.total_pos = p.N * Hg * Wg;
            { const int ti_ = 0; t.wtap[ti_] = 0; t.shift[ti_] = 0; } t.gbeg[1] = 1;
            if (!encode_flat(&tp.map_a, act, chan_a, t.total_pos)) return 0;
            if (p.stride == 2 && !p.out_compact) { t.dense = 0; t.OH = p.H; t.OW = p.W; t.os = 2; out_pixels = (long long)p.N * p.H * p.W; }   // scattered to the even positions
            else { t.dense = 1; t.OH = Hg; t.OW = Wg; out_pixels = t.total_pos; }
        } else if (p.ksz == 1) {
            // forward of a stride-2 1x1 layer: the positions are the output pixels, the window gathers every second input pixel
            Tall g; if (!tall_of(p.P, p.Q, 0, 2, g)) return 0;
            t.a_flat = 0; t.dense = 1; t.es = 2; t.Hp = g.Hp; t.Wp = g.Wp; t.R = g.R; t.box_pos = g.box_pos; t.a_box_bytes = g.box_bytes; t.hb = 0;
            t.nbox = boxes_for(TILE_M, g.box_pos); t.total_pos = p.N * g.Hp * g.Wp; t.OH = p.P; t.OW = p.Q; out_pixels = t.total_pos;
            { const int ti_ = 0; t.wtap[ti_] = 0; t.shift[ti_] = 0; } t.gbeg[1] = 1;
            if (!encode_tall(&tp.map_a, act, chan_a, p.N, p.H, p.W, g.Wp, g.box_h, g.box_n, 2)) return 0;
        } else if (p.stride == 1) {
            // 3x3 at stride 1: one window, nine taps; dgrad walks the taps mirrored
            Tall g; if (!tall_of(p.H, p.W, 1, 1, g)) return 0;
            t.a_flat = 0; t.dense = 0; t.pad = 1; t.Hp = g.Hp; t.Wp = g.Wp; t.R = g.R; t.box_pos = g.box_pos; t.a_box_bytes = g.box_bytes; t.hb = g.Wp + 1;
            t.nbox = boxes_for(TILE_M + 2 * t.hb, g.box_pos); t.total_pos = p.N * g.Hp * g.Wp; t.OH = p.H; t.OW = p.W; out_pixels = (long long)p.N * p.H * p.W;
            for (int w = 0; w < 9; ++w) { const int ti_ = w; t.wtap[ti_] = mode == CONV_DGRAD ? 8 - w : w; t.shift[ti_] = (w / 3) * g.Wp + (w % 3); }
            t.gbeg[1] = 9;
            if (!encode_tall(&tp.map_a, act, chan_a, p.N, p.H, p.W, g.Wp, g.box_h, g.box_n, 1)) return 0;
        } else if (mode == CONV_FWD) {
            // 3x3 at stride 2, forward: positions over the P x Q outputs, one window per input parity phase (element-strided fetch)
            Tall g; if (!tall_of(p.P, p.Q, 1, 2, g)) return 0;
            t.a_flat = 0; t.dense = 0; t.pad = 1; t.es = 2; t.Hp = g.Hp; t.Wp = g.Wp; t.R = g.R; t.box_pos = g.box_pos; t.a_box_bytes = g.box_bytes; t.hb = g.Wp + 1;
            t.nbox = boxes_for(TILE_M + t.hb, g.box_pos); t.total_pos = p.N * g.Hp * g.Wp; t.OH = p.P; t.OW = p.Q; out_pixels = (long long)p.N * p.P * p.Q;
            int n = 0; t.ngroups = 0;
            for (int u = 0; u < 2; ++u) for (int v = 0; v < 2; ++v) {
                int rs[4][2]; const int k = phase_taps(u, v, rs);
                t.gxs[t.ngroups] = v; t.gys[t.ngroups] = u;
                for (int i = 0; i < k; ++i) {
                    const int di = rs[i][0] == 0 ? -1 : 0, dj = rs[i][1] == 0 ? -1 : 0;    // tap 0 reads the previous phase row / column
                    { const int ti_ = n++; t.wtap[ti_] = rs[i][0] * 3 + rs[i][1]; t.shift[ti_] = t.hb + di * g.Wp + dj; }
                }
                t.gbeg[++t.ngroups] = n;
            }
            if (!encode_tall(&tp.map_a, act, chan_a, p.N, p.H, p.W, g.Wp, g.box_h, g.box_n, 2)) return 0;
        } else {
            // 3x3 at stride 2, dgrad: one problem per output parity phase (u, v), positions over the P x Q grid of dy; input row 2i + u
            // takes dy row i + (u + 1 - r) / 2 through tap r
            const int u = ph >> 1, v = ph & 1;
            Tall g; if (!tall_of(p.P, p.Q, 1, 1, g)) return 0;
            t.a_flat = 0; t.dense = 0; t.pad = 1; t.Hp = g.Hp; t.Wp = g.Wp; t.R = g.R; t.box_pos = g.box_pos; t.a_box_bytes = g.box_bytes; t.hb = 0;
            t.nbox = boxes_for(TILE_M + g.Wp + 1, g.box_pos); t.total_pos = p.N * g.Hp * g.Wp;
            t.OH = p.H; t.OW = p.W; t.os = 2; t.oy = u; t.ox = v; out_pixels = (long long)p.N * p.H * p.W;
            int rs[4][2]; const int k = phase_taps(u, v, rs);
            for (int i = 0; i < k; ++i) { const int ti_ = i; t.wtap[ti_] = rs[i][0] * 3 + rs[i][1]; t.shift[ti_] = ((u + 1 - rs[i][0]) / 2) * g.Wp + (v + 1 - rs[i][1]) / 2; }
            t.gbeg[1] = k;
            if (!encode_tall(&tp.map_a, act, chan_a, p.N, p.P, p.Q, g.Wp, g.box_h, g.box_n, 1)) return 0;
        }
        // residual
        t.add_mode = !p.add ? 0 : p.add_sub == 2 ? 3 : 2;
        // output tiles: up to 256 columns, a multiple of 64 when there are several
        const int n_cap = 256;
        const int ntaps = t.gbeg[t.ngroups];
        auto b_tile = [&](int nt) { return mode == CONV_FWD ? nt * 128 : ((nt + 63) / 64) * 8192; };
        auto b_total = [&](int nt) { return (size_t)t.slabs * ntaps * ((b_tile(nt) + 1023) / 1024 * 1024); };
        t.tiles_n = (ncol + n_cap - 1) / n_cap;
        t.n_tile = (ncol + t.tiles_n - 1) / t.tiles_n;
        t.n_tile = t.tiles_n > 1 ? (t.n_tile + 63) / 64 * 64 : (t.n_tile + 15) / 16 * 16;
        t.tiles_n = (ncol + t.n_tile - 1) / t.n_tile;
        t.out_slabs = (t.n_tile + 63) / 64;
        t.tiles_m = (t.total_pos + TILE_M - 1) / TILE_M;
        t.b_bytes = b_tile(t.n_tile);
        t.b_total = (int)b_total(t.n_tile);
        // weights [K][taps][C] viewed as (C, tap, K).  Forward: a tile is n_tile output channels (rows) x 64 input channels.
        // dgrad: a block is 64 reduction channels k (rows) x 64 output columns c.
        { const uint64_t dims[3] = {(uint64_t)p.C, (uint64_t)taps, (uint64_t)p.K};
          const uint64_t st[2] = {(uint64_t)p.C * 2, (uint64_t)taps * p.C * 2};
          const uint32_t box[3] = {64, 1, mode == CONV_FWD ? (uint32_t)t.n_tile : 64u};
          if (!encode_map(&tp.map_b, p.wgt, 3, dims, st, box)) return 0; }
        if (t.dense) {
            if (!encode_flat(&tp.map_out, p.out, ncol, out_pixels)) return 0;
        }
        memcpy((char*)host_tc + (size_t)ph * sizeof(TcProb), &tp, sizeof(tp));
    }
    return count;
}
size_t conv_tc_prob_bytes() { return sizeof(TcProb); }
// units of work of a problem: pairs of row tiles x column tiles
int conv_tc_tiles(const void* host_tc) { const TcHot* t = &((const TcProb*)host_tc)->h; return ((t->tiles_m + 1) / 2) * t->tiles_n; }
// packs what a launch has to know about its largest problem into one number: window KB (12 bits), weight-tile KB (12), staging
// tiles (4), KB of all weight tiles of a column tile (16), MMA N (20)
size_t conv_tc_smem(const void* host_tc) {
    const TcHot* t = &((const TcProb*)host_tc)->h;
    const size_t a_stage = ((size_t)t->nbox * t->a_box_bytes + 1023) / 1024, b_stage = ((size_t)t->b_bytes + 1023) / 1024;
    return (a_stage << 52) | (b_stage << 40) | ((size_t)(t->add_mode == 1 ? 2 : 1) << 36) | ((size_t)std::min(t->b_total / 1024, 0xFFFF) << 20) | (size_t)t->n_tile;
}
// field-wise maximum of two packed values
size_t conv_tc_merge(size_t a, size_t b) {
    return (std::max(a >> 52, b >> 52) << 52) | (std::max((a >> 40) & 0xFFF, (b >> 40) & 0xFFF) << 40) | (std::max((a >> 36) & 0xF, (b >> 36) & 0xF) << 36) |
           (std::max((a >> 20) & 0xFFFF, (b >> 20) & 0xFFFF) << 20) | std::max(a & 0xFFFFF, b & 0xFFFFF);
}

constexpr size_t TC_SMEM_BUDGET = 204 * 1024;

// total_tiles: an upper bound of the tiles of all problems of the launch (max_tiles * nprob); packed: conv_tc_merge over its problems
void launch_conv_tc_probs(const void* d_tc, int nprob, int max_tiles, size_t packed, cudaStream_t s) {
    static bool configured = false; static int sms = 0;
    if (!configured) {
        cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(TC_SMEM_BUDGET + 1024));
        int dev = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        configured = true;
    }
    TcLaunch L{};
    L.nprob = nprob;
    L.a_stage = (int)(packed >> 52) * 1024; L.b_stage = (int)((packed >> 40) & 0xFFF) * 1024;
    const int n_tile = (int)(packed & 0xFFFFF);
    // Shared memory.  Two epilogue groups, each with two 16 KB slab buffers (one where the rings need the room).  The windows' ring
    // gets four stages (two pairs of tiles), the weights' ring what is left, up to eight tiles; any rest goes back to the windows.
    // A layer runs at the bytes it keeps in flight.
    const size_t a = (size_t)L.a_stage, b = (size_t)L.b_stage;
    L.groups = 2; L.pg = 2;
    if ((size_t)L.groups * L.pg * SLAB_BYTES + 4 * a + 3 * b > TC_SMEM_BUDGET) L.pg = 1;
    const size_t rings = TC_SMEM_BUDGET - (size_t)L.groups * L.pg * SLAB_BYTES;
    L.na = 4; while (L.na > 2 && (size_t)L.na * a + 2 * b > rings) --L.na;
    L.nb = 2; while (L.nb < 8 && (size_t)L.na * a + (size_t)(L.nb + 1) * b <= rings) ++L.nb;
    while (L.na < TC_MAX_STAGES && (size_t)(L.na + 1) * a + (size_t)L.nb * b <= rings) ++L.na;
    L.acc_stride = (n_tile + 31) / 32 * 32;
    L.nbuf = L.acc_stride <= 128 ? 2 : 1;
    L.tmem_cols = 32; while (L.tmem_cols < 2 * L.nbuf * L.acc_stride) L.tmem_cols *= 2;
    // at least 120 KB of shared memory so that two CTAs that allocate tensor memory never share an SM
    const size_t smem = std::max((size_t)L.na * a + (size_t)L.nb * b + (size_t)L.groups * L.pg * SLAB_BYTES, (size_t)120 * 1024) + 1024;
    const long long total = (long long)max_tiles * nprob;
    const int grid = (int)std::max(1ll, std::min(total, (long long)sms));
    conv_tc_kernel<<<grid, TC_CONV_THREADS, smem, s>>>((const TcProb*)d_tc, L);
}

// ---- wgrad host side
struct WgGeom { TcWgradProb t; size_t smem, partial_bytes; int box_h, box_n; };

static bool wg_geometry_box(const ConvProb& p, int target_ctas, WgGeom& w, int max_box);
// Both operands of a 3x3 weight gradient are windows of boxes, so a stage is large and the boxes' rounding decides how many stages
// fit: the largest boxes that still leave two stages are taken (fewer TMA issues), else the size with the most stages.
static bool wg_geometry(const ConvProb& p, int target_ctas, WgGeom& w) {
    if (p.ksz == 1) return wg_geometry_box(p, target_ctas, w, 96);
    const int caps[5] = {96, 64, 48, 32, 24};
    WgGeom best; int best_stages = 0;
    for (int i = 0; i < 5; ++i) {
        WgGeom g;
        if (!wg_geometry_box(p, target_ctas, g, caps[i])) continue;
        if (g.t.stages > best_stages) { best = g; best_stages = g.t.stages; }
        if (best_stages >= 2) break;
    }
    if (!best_stages) return false;
    w = best;
    return true;
}
static bool wg_geometry_box(const ConvProb& p, int target_ctas, WgGeom& w, int max_box) {
    if (!tc_shape_ok(p)) return false;
    if (((uintptr_t)p.act | (uintptr_t)p.wgt) & 15) return false;
    TcWgradProb& t = w.t; memset(&t, 0, sizeof(t));
    const int taps = p.ksz * p.ksz;
    t.taps = taps; t.n_img = p.N; t.cout = p.K; t.cin = p.C; t.es = 1; t.pad = 0;
    long long total_pos;
    if (p.ksz == 1 && p.stride == 1) {
        t.dy_flat = 1; t.a_flat = 1; t.Hp = p.H; t.Wp = p.W; t.box_pos = TILE_M; t.nbox_dy = 1; t.nbox_a = 1; t.hb = 0;
        t.dy_box_bytes = SLAB_BYTES; t.a_box_bytes = SLAB_BYTES; total_pos = (long long)p.N * p.H * p.W;
        t.tap_groups = 1; t.gbeg[1] = 1; t.tap[0] = TapRef{0, 0};
    } else if (p.ksz == 1) {
        // stride-2 1x1: the positions are the P x Q pixels of dy in order; a is gathered at every second pixel
        Tall g; if (!tall_of(p.P, p.Q, 0, 2, g)) return false;
        w.box_h = g.box_h; w.box_n = g.box_n;
        t.dy_flat = 1; t.a_flat = 0; t.es = 2; t.Hp = g.Hp; t.Wp = g.Wp; t.R = g.R; t.box_pos = g.box_pos; t.hb = 0;
        t.nbox_dy = 1; t.dy_box_bytes = SLAB_BYTES; t.nbox_a = boxes_for(TILE_M, g.box_pos); t.a_box_bytes = g.box_bytes;
        total_pos = (long long)p.N * g.Hp * g.Wp;
        t.tap_groups = 1; t.gbeg[1] = 1; t.tap[0] = TapRef{0, 0};
    } else if (p.stride == 1) {
        Tall g; if (!tall_of(p.H, p.W, 1, 1, g, max_box)) return false;
        w.box_h = g.box_h; w.box_n = g.box_n;
        t.dy_flat = 0; t.a_flat = 0; t.pad = 1; t.Hp = g.Hp; t.Wp = g.Wp; t.R = g.R; t.box_pos = g.box_pos; t.hb = g.Wp + 1;
        t.nbox_dy = boxes_for(TILE_M, g.box_pos); t.nbox_a = boxes_for(TILE_M + 2 * t.hb, g.box_pos); t.dy_box_bytes = g.box_bytes; t.a_box_bytes = g.box_bytes;
        total_pos = (long long)p.N * g.Hp * g.Wp;
        for (int i = 0; i < 9; ++i) t.tap[i] = TapRef{i, (i / 3) * g.Wp + (i % 3)};
        t.tap_groups = 0;                                // groups of up to three taps: set below, once the column tile is known
    } else {
        Tall g; if (!tall_of(p.P, p.Q, 1, 2, g, max_box)) return false;
        Tall gd; if (!tall_of(p.P, p.Q, 1, 1, gd, max_box)) return false;
        if (gd.R != g.R || gd.Hp != g.Hp) return false;          // both operands walk the same boxes of rows
        w.box_h = g.box_h; w.box_n = g.box_n;
        t.dy_flat = 0; t.a_flat = 0; t.pad = 1; t.es = 2; t.Hp = g.Hp; t.Wp = g.Wp; t.R = g.R; t.box_pos = g.box_pos; t.hb = g.Wp + 1;
        t.nbox_dy = boxes_for(TILE_M, g.box_pos); t.nbox_a = boxes_for(TILE_M + t.hb, g.box_pos); t.dy_box_bytes = g.box_bytes; t.a_box_bytes = g.box_bytes;
        total_pos = (long long)p.N * g.Hp * g.Wp;
        int n = 0; t.tap_groups = 0;
        for (int u = 0; u < 2; ++u) for (int v = 0; v < 2; ++v) {
            int rs[4][2]; const int k = phase_taps(u, v, rs);
            t.gxs[t.tap_groups] = v; t.gys[t.tap_groups] = u;
            for (int i = 0; i < k; ++i) t.tap[n++] = TapRef{rs[i][0] * 3 + rs[i][1], t.hb + (rs[i][0] == 0 ? -1 : 0) * g.Wp + (rs[i][1] == 0 ? -1 : 0)};
            t.gbeg[++t.tap_groups] = n;
        }
    }
    t.chunks = (int)((total_pos + TILE_M - 1) / TILE_M);
    t.m_tiles = (p.K + 127) / 128;
    // columns of one CTA: the input channels in tiles of at most 256 (1x1) or 128 (3x3: up to four taps in 512 columns of tensor memory)
    const int n_cap = taps == 1 ? 256 : 128;
    t.n_tiles = (p.C + n_cap - 1) / n_cap;
    t.n_tile = (p.C + t.n_tiles - 1) / t.n_tiles;
    t.n_tile = t.n_tiles > 1 ? (t.n_tile + 63) / 64 * 64 : (t.n_tile + 15) / 16 * 16;
    t.n_tiles = (p.C + t.n_tile - 1) / t.n_tile;
    t.a_slabs = (t.n_tile + 63) / 64;
    if (taps == 9 && p.stride == 1) { for (int g = 0; g < 3; ++g) { t.gbeg[g + 1] = 3 * (g + 1); t.gxs[g] = 0; t.gys[g] = 0; } t.tap_groups = 3; }
    int max_group = 0; for (int g = 0; g < t.tap_groups; ++g) max_group = std::max(max_group, t.gbeg[g + 1] - t.gbeg[g]);
    int max_acc = 0; for (int g = 0; g < t.tap_groups; ++g) { const int n = t.gbeg[g + 1] - t.gbeg[g]; max_acc = std::max(max_acc, n + (n & 1)); }   // an odd group's last tap takes two accumulators
    (void)max_group;
    t.tmem_cols = 32; while (t.tmem_cols < max_acc * t.n_tile) t.tmem_cols *= 2;
    if (t.tmem_cols > 512) return false;
    t.dy_slab_bytes = (t.nbox_dy * t.dy_box_bytes + 1023) / 1024 * 1024;
    t.a_slab_bytes = (t.nbox_a * t.a_box_bytes + 1023) / 1024 * 1024;
    t.stage_bytes = 2 * t.dy_slab_bytes + t.a_slabs * t.a_slab_bytes;
    t.stages = TC_MAX_STAGES; while (t.stages > 1 && (size_t)t.stages * t.stage_bytes > TC_SMEM_BUDGET) --t.stages;
    if ((size_t)t.stages * t.stage_bytes > TC_SMEM_BUDGET) return false;
    w.smem = std::max((size_t)t.stages * t.stage_bytes, (size_t)120 * 1024) + 1024;
    // Split of the positions.  target_ctas is twice this problem's share of the SMs.  Every CTA pays a fixed cost (set-up, the
    // accumulators' way out) worth about six chunks, and a launch takes whole waves, so the split is the one that minimises
    // waves x (chunks per CTA + 6): mostly one full wave.  The partial buffer is sized for the most splits any share could pick.
    const int fixed = t.m_tiles * t.n_tiles * t.tap_groups;
    const int want_max = std::max(1, std::min(std::min(t.chunks, 256), target_ctas / fixed));
    const int share = std::max(1, target_ctas / 2);
    long long best_cost = -1; int best_cps = t.chunks;
    for (int sp = 1; sp <= want_max; ++sp) {
        const int cps = (t.chunks + sp - 1) / sp, eff = (t.chunks + cps - 1) / cps;
        const long long waves = ((long long)fixed * eff + share - 1) / share, cost = waves * (cps + 6);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_cps = cps; }
    }
    t.chunks_per_split = best_cps; t.splits = (t.chunks + best_cps - 1) / best_cps;
    w.partial_bytes = want_max > 1 ? (size_t)want_max * taps * p.K * p.C * 4 : 0;
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
    TcWgradProb& t = g.t;
    if (t.dy_flat) { if (!encode_flat(&t.map_dy, p.wgt, p.K, (long long)p.N * p.P * p.Q)) return false; }
    else if (!encode_tall(&t.map_dy, p.wgt, p.K, p.N, p.P, p.Q, t.Wp, g.box_h, g.box_n, 1)) return false;
    if (t.a_flat) { if (!encode_flat(&t.map_a, p.act, p.C, (long long)p.N * p.H * p.W)) return false; }
    else if (!encode_tall(&t.map_a, p.act, p.C, p.N, p.H, p.W, t.Wp, g.box_h, g.box_n, t.es)) return false;
    t.partial = p.partial; t.out = (float*)p.out; t.status = conv_tc_status_word();
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
