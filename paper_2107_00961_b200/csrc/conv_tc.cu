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

constexpr int TC_THREADS = 192;              // wgrad kernel: producer warp, MMA warp, four epilogue warps
constexpr int TC_CONV_THREADS = 320;         // forward / dgrad kernel: producer warp, MMA warp, two groups of four epilogue warps
constexpr int TC_MAX_STAGES = 12;
constexpr int TILE_M = 128;
constexpr int SLAB_BYTES = TILE_M * 128;      // 128 rows x 64 channels of bf16
constexpr size_t TC_RESIDENT_BUDGET = 96 * 1024;   // weights of one column tile that may stay in shared memory

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
    int add_mode;             // 0 none; 1 fetched by TMA into the staging tile (dense); 2 global loads at the output pixel; 3 global loads from a compact tensor that applies at even (y, x) only
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
    CUtensorMap map_add;      // dense problems with a residual: the residual likewise
    TcHot h;
};
static_assert(sizeof(TcHot) % 4 == 0, "copied word by word");

struct TcLaunch { int nprob, na, nb, a_stage, b_stage, tmem_cols, acc_stride, n_stg, stg_bytes, b_res, b_region, groups, pg, prefetch; };   // b_res: the weights of a (problem, column tile) stay in shared memory; b_region: bytes of the weight ring or of the resident weights;
// groups: epilogue groups (they take alternate tiles); pg: staging tiles per group (n_stg = groups * pg); prefetch: some problem's residual is fetched by TMA
constexpr int TC_MAX_PROBS = 128;             // descriptors per launch (sub-ResNets x output phases)

__device__ __forceinline__ void copy_hot(TcHot* dst, const TcHot* src, int tid, int nthreads) {
    const uint32_t* s4 = reinterpret_cast<const uint32_t*>(src); uint32_t* d4 = reinterpret_cast<uint32_t*>(dst);
    for (int i = tid; i < (int)(sizeof(TcHot) / 4); i += nthreads) d4[i] = __ldg(s4 + i);
}

__global__ void __launch_bounds__(TC_CONV_THREADS, 1) conv_tc_kernel(const TcProb* __restrict__ probs, const TcLaunch L) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bars[4 * TC_MAX_STAGES + 14];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int pix_s2[2][TILE_M];
    __shared__ float stat_s2[2][4][2][256];
    __shared__ int tile_end_s[TC_MAX_PROBS];                      // running sum of the problems' tile counts
    __shared__ TcHot hot_s[4];                                    // the current problem of the producer, the MMA issuer, the two epilogue groups
    const uint32_t a_full = smem_u32(&bars[0]), a_empty = smem_u32(&bars[TC_MAX_STAGES]);
    const uint32_t b_full = smem_u32(&bars[2 * TC_MAX_STAGES]), b_empty = smem_u32(&bars[3 * TC_MAX_STAGES]);
    const uint32_t acc_full = smem_u32(&bars[4 * TC_MAX_STAGES]), acc_empty = smem_u32(&bars[4 * TC_MAX_STAGES + 2]);
    const uint32_t add_full = smem_u32(&bars[4 * TC_MAX_STAGES + 4]), stg_free = smem_u32(&bars[4 * TC_MAX_STAGES + 8]);
    const uint32_t bres_full = smem_u32(&bars[4 * TC_MAX_STAGES + 12]), bres_empty = smem_u32(&bars[4 * TC_MAX_STAGES + 13]);
    const uint32_t a_ring = smem_u32(smem), b_ring = a_ring + (uint32_t)(L.na * L.a_stage), stg_base = b_ring + (uint32_t)L.b_region;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) {
            mbar_init(a_full + 8 * s, 1); mbar_init(a_empty + 8 * s, 1); mbar_init(b_full + 8 * s, 1); mbar_init(b_empty + 8 * s, 1);
        }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full + 8 * s, 1); mbar_init(acc_empty + 8 * s, 4); }
        for (int s = 0; s < 4; ++s) { mbar_init(add_full + 8 * s, 1); mbar_init(stg_free + 8 * s, 1); }
        mbar_init(bres_full, 1); mbar_init(bres_empty, 1);
        abort_s = 0;
        int run = 0;
        for (int i = 0; i < L.nprob; ++i) { run += probs[i].h.tiles_m * probs[i].h.tiles_n; tile_end_s[i] = run; }
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
    // The tiles of all problems, column tile innermost, are dealt round-robin: the CTAs that run side by side work on neighbouring
    // tiles, share activation windows and weight tiles in L2 and read HBM as one moving front.  (Contiguous runs per CTA, with the
    // column tile outermost, were measured too: no faster, and slower for the layers whose weights stream.)
    const int t_begin = (int)blockIdx.x, t_stop = tile_end_s[L.nprob - 1], t_step = (int)gridDim.x;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t a_cnt = 0, b_cnt = 0, seq = 0, add_use[4] = {0u, 0u, 0u, 0u}; bool ok = true;
            int cur = -1; TcHot& h = hot_s[0];
            int sa = 0, sb_ = 0; uint32_t pha = 0, phb = 0;       // ring positions and phases
            int cur_unit = -1; uint32_t unit_cnt = 0;
            for (int t = t_begin; t < t_stop && ok; t += t_step, ++seq) {
                int pi = 0; while (t >= tile_end_s[pi]) ++pi;
                if (pi != cur) { copy_hot(&h, &probs[pi].h, 0, 1); cur = pi; }
                const TcProb* pp = probs + pi;
                const int loc = t - (pi ? tile_end_s[pi - 1] : 0);
                const int n_tile = h.n_tile, slabs = h.slabs, ngroups = h.ngroups, a_flat = h.a_flat, nbox = h.nbox,
                          a_box_bytes = h.a_box_bytes, R = h.R, Hp = h.Hp, pad = h.pad, es = h.es, b_bytes = h.b_bytes, mn = h.b_mn_major;
                const int tiles_n = h.tiles_n, tn = loc % tiles_n, tm = loc / tiles_n;
                if (L.b_res && (pi << 8 | tn) != cur_unit) {
                    // new (problem, column tile): all its weight tiles go to the resident region, once the MMAs of the last one have read theirs
                    if (!mbar_wait(bres_empty, (unit_cnt & 1u) ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 8); ok = false; break; }
                    const int ntaps = h.gbeg[ngroups];
                    mbar_expect_tx(bres_full, (uint32_t)(slabs * ntaps * b_bytes));
                    for (int sl = 0; sl < slabs; ++sl)
                        for (int tap = 0; tap < ntaps; ++tap) {
                            const uint32_t dst = b_ring + (uint32_t)((sl * ntaps + tap) * ((b_bytes + 1023) & ~1023));
                            const int wtap = h.wtap[tap];
                            if (!mn) tma_load_3d(dst, &pp->map_b, bres_full, sl * 64, wtap, tn * n_tile);
                            else for (int j = 0; j * 64 < n_tile; ++j)
                                tma_load_3d(dst + (uint32_t)(j * 8192), &pp->map_b, bres_full, tn * n_tile + j * 64, wtap, sl * 64);
                        }
                    ++unit_cnt; cur_unit = pi << 8 | tn;
                }
                if (h.add_mode == 1) {
                    // the residual tile goes straight into the staging tile the epilogue will finish in place
                    const uint32_t grp = L.groups == 2 ? (seq & 1u) : 0u, kk = L.groups == 2 ? (seq >> 1) : seq;
                    const uint32_t sb = grp * (uint32_t)L.pg + kk % (uint32_t)L.pg, uses = kk / (uint32_t)L.pg;
                    if (!mbar_wait(stg_free + 8 * sb, (uses & 1u) ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 7); ok = false; break; }
                    mbar_expect_tx(add_full + 8 * sb, (uint32_t)(h.out_slabs * SLAB_BYTES));
                    for (int j = 0; j < h.out_slabs; ++j)
                        tma_load_2d(stg_base + sb * (uint32_t)L.stg_bytes + (uint32_t)(j * SLAB_BYTES), &pp->map_add, add_full + 8 * sb, tn * n_tile + j * 64, tm * TILE_M);
                    ++add_use[sb];
                }
                const int bx0 = a_flat ? 0 : floor_div(tm * TILE_M - h.hb, h.box_pos);
                for (int sl = 0; sl < slabs && ok; ++sl) {
                    for (int g = 0; g < ngroups && ok; ++g) {
                        {
                            if (!mbar_wait(a_empty + 8 * sa, pha ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 1); ok = false; break; }
                            const uint32_t dst = a_ring + (uint32_t)(sa * L.a_stage);
                            mbar_expect_tx(a_full + 8 * sa, (uint32_t)(nbox * a_box_bytes));
                            if (a_flat) tma_load_2d(dst, &pp->map_a, a_full + 8 * sa, sl * 64, tm * TILE_M);
                            else {
                                const int gx = h.gxs[g], gy = h.gys[g];
                                for (int i = 0; i < nbox; ++i) {
                                    const int trow = (bx0 + i) * R, img = floor_div(trow, Hp), yy0 = trow - img * Hp;
                                    tma_load_4d(dst + (uint32_t)(i * a_box_bytes), &pp->map_a, a_full + 8 * sa, sl * 64, gx, (yy0 - pad) * es + gy, img);
                                }
                            }
                            ++a_cnt; if (++sa == L.na) { sa = 0; pha ^= 1u; }
                        }
                        const int t_end = L.b_res ? 0 : h.gbeg[g + 1];
                        for (int tap = h.gbeg[g]; tap < t_end; ++tap) {
                            if (!mbar_wait(b_empty + 8 * sb_, phb ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 2); ok = false; break; }
                            const uint32_t dst = b_ring + (uint32_t)(sb_ * L.b_stage);
                            const int wtap = h.wtap[tap];
                            mbar_expect_tx(b_full + 8 * sb_, (uint32_t)b_bytes);
                            if (!mn) tma_load_3d(dst, &pp->map_b, b_full + 8 * sb_, sl * 64, wtap, tn * n_tile);
                            else for (int j = 0; j * 64 < n_tile; ++j)
                                tma_load_3d(dst + (uint32_t)(j * 8192), &pp->map_b, b_full + 8 * sb_, tn * n_tile + j * 64, wtap, sl * 64);
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
                for (uint32_t sb = 0; sb < 4; ++sb)
                    if (add_use[sb]) for (int i = 0; i < 4096 && !mbar_try(add_full + 8 * sb, (add_use[sb] - 1u) & 1u); ++i) __nanosleep(64);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t acc_cnt = 0; bool ok = true;
            int cur = -1; TcHot& h = hot_s[1];
            int sa = 0, sb = 0; uint32_t pha = 0, phb = 0;
            int cur_unit = -1; uint32_t unit_cnt = 0;
            // the constant part of a 128-byte-swizzle descriptor: stride between 8-row groups 1024 bytes, version, swizzle mode
            const uint64_t desc_k = desc_sw128(0, 16, 1024), desc_mn = desc_sw128(0, 8192, 1024);
            for (int t = t_begin; t < t_stop && ok; t += t_step, ++acc_cnt) {
                int pi = 0; while (t >= tile_end_s[pi]) ++pi;
                if (pi != cur) { copy_hot(&h, &probs[pi].h, 0, 1); cur = pi; }
                const int loc = t - (pi ? tile_end_s[pi - 1] : 0);
                const int slabs = h.slabs, ngroups = h.ngroups, red = h.red, mn = h.b_mn_major;
                const int tiles_n = h.tiles_n, tn = loc % tiles_n, tm = loc / tiles_n;
                const int ntaps = h.gbeg[ngroups], b_stride = (h.b_bytes + 1023) & ~1023;
                if (L.b_res && (pi << 8 | tn) != cur_unit) {
                    if (!mbar_wait(bres_full, unit_cnt & 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 9); ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    ++unit_cnt; cur_unit = pi << 8 | tn;
                }
                const int bx0 = h.a_flat ? 0 : floor_div(tm * TILE_M - h.hb, h.box_pos);
                const int a_off = h.a_flat ? 0 : tm * TILE_M - h.hb - bx0 * h.box_pos;
                const uint32_t buf = acc_cnt & 1u, aph = (acc_cnt >> 1) & 1u;
                if (!mbar_wait(acc_empty + 8 * buf, aph ^ 1u, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 3); ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
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
                        if (!mbar_wait(a_full + 8 * sa, pha, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 4); ok = false; break; }
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint32_t a_rows16 = ((a_ring + (uint32_t)(sa * L.a_stage)) >> 4) + (uint32_t)a_off * 8u;   // start address in 16-byte units
                        const int t_end = h.gbeg[g + 1];
                        for (int tap = h.gbeg[g]; tap < t_end; ++tap) {
                            const uint32_t a16 = a_rows16 + (uint32_t)h.shift[tap] * 8u;
                            uint32_t b16;
                            if (L.b_res) b16 = (b_ring + (uint32_t)((sl * ntaps + tap) * b_stride)) >> 4;
                            else {
                                if (!mbar_wait(b_full + 8 * sb, phb, &abort_s)) { atomicExch(&abort_s, 1); atomicExch(h.status, 5); ok = false; break; }
                                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                                b16 = (b_ring + (uint32_t)(sb * L.b_stage)) >> 4;
                            }
                            for (int k16 = 0; k16 < ksteps; ++k16) {
                                umma_bf16(d_tmem, desc_k | (uint64_t)((a16 + 2u * (uint32_t)k16) & 0x3FFFu), b_const | (uint64_t)((b16 + b_step * (uint32_t)k16) & 0x3FFFu), idesc, acc);
                                acc = 1;
                            }
                            if (!L.b_res) {
                                umma_commit(b_empty + 8 * sb);   // weight tile reusable once these MMAs have read it
                                if (++sb == L.nb) { sb = 0; phb ^= 1u; }
                            }
                        }
                        umma_commit(a_empty + 8 * sa);
                        if (++sa == L.na) { sa = 0; pha ^= 1u; }
                    }
                }
                if (ok) umma_commit(acc_full + 8 * buf);         // accumulator complete
                if (ok && L.b_res) {
                    // last tile of this (problem, column tile) for this CTA: the resident weights may be replaced once these MMAs are done
                    bool last = t + t_step >= t_stop;
                    if (!last) { const int t2 = t + t_step; int pn = pi; while (t2 >= tile_end_s[pn]) ++pn; const int l2 = t2 - (pn ? tile_end_s[pn - 1] : 0);
                        last = pn != pi || l2 % tiles_n != tn; }
                    if (last) umma_commit(bres_empty);
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue: two groups of 4 warps (one TMEM lane quadrant each);
        // group g takes the tiles whose accumulator is buffer g, so two epilogues run side by side
        const int grp = (warp - 2) >> 2, bid = 1 + grp;
        const int quad = warp & 3;
        const int m = quad * 32 + lane;                          // row of the tile = TMEM lane
        const int et = threadIdx.x - 64 - grp * 128;             // 0..127 among the group's threads
        const bool leader = et == 0;
        int* const pix_s = pix_s2[grp];
        float (*const stat_s)[2][256] = stat_s2[grp];
        uint32_t add_use[4] = {0u, 0u, 0u, 0u}; bool ok = true;
        int cur = -1; const TcHot& h = hot_s[2 + grp];
        for (int t = t_begin + grp * t_step; grp < L.groups && t < t_stop && ok; t += L.groups * t_step) {
            const uint32_t acc_cnt = (uint32_t)((t - t_begin) / t_step), kk = acc_cnt / (uint32_t)L.groups;     // tile number of the CTA, of the group
            int pi = 0; while (t >= tile_end_s[pi]) ++pi;
            const TcProb* pp = probs + pi;
            const int loc = t - (pi ? tile_end_s[pi - 1] : 0);
            const uint32_t buf = acc_cnt & 1u, aph = (acc_cnt >> 1) & 1u;
            const uint32_t sb = (uint32_t)(grp * L.pg) + kk % (uint32_t)L.pg;
            const uint32_t stg = stg_base + sb * (uint32_t)L.stg_bytes;
            if (leader) {
                // the staging tile of this tile (and, with a prefetched residual, the next tile's, which the producer is waiting to
                // fill) must have been read by the bulk store issued from it
                bulk_wait_read(L.prefetch ? L.pg - 2 : L.pg - 1);
                if (L.prefetch && kk + 1 >= (uint32_t)L.pg) mbar_arrive(stg_free + 8 * ((uint32_t)(grp * L.pg) + (kk + 1) % (uint32_t)L.pg));
            }
            // ... and every warp must have finished its share of the last copy-out
            bar_sync_epi(bid);
            if (pi != cur) { copy_hot(&hot_s[2 + grp], &probs[pi].h, et, 128); cur = pi; bar_sync_epi(bid); }
            const int n_tile = h.n_tile, ncol = h.ncol, add_mode = h.add_mode, dense = h.dense, out_slabs = h.out_slabs;
            const float scale = h.scale;
            const __nv_bfloat16* addp = h.add; __nv_bfloat16* outp = h.out; float* stat_tiles = h.stat_tiles;
            const int tiles_n = h.tiles_n, tn = loc % tiles_n, tm = loc / tiles_n;
            ok = mbar_wait(acc_full + 8 * buf, aph, &abort_s);
            if (ok && add_mode == 1) { ok = mbar_wait(add_full + 8 * sb, add_use[sb] & 1u, &abort_s); ++add_use[sb]; }
            ok = bar_and_epi(bid, ok);                           // one decision for the four warps: they share the barriers below
            if (!ok) { atomicExch(&abort_s, 1); atomicExch(h.status, 6); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
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
            const uint32_t t_row = tmem_base + buf * (uint32_t)L.acc_stride + ((uint32_t)(quad * 32) << 16);
            const int col0 = tn * n_tile;
            const uint32_t s_row = stg + (uint32_t)m * 128u;
            const bool gadd = add_mode >= 2 && valid && addpix >= 0;
            for (int c0 = 0; c0 < n_tile; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(t_row + (uint32_t)c0, v);
                uint4 ga[4];
                if (gadd) {
#pragma unroll
                    for (int g = 0; g < 4; ++g)
                        ga[g] = (c0 + g * 8 < n_tile && col0 + c0 + g * 8 < ncol) ? __ldg(reinterpret_cast<const uint4*>(addp + addpix * ncol + col0 + c0 + g * 8)) : make_uint4(0u, 0u, 0u, 0u);
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int c = c0 + g * 8;
                    if (c < n_tile) {
                        const uint32_t sa = s_row + (uint32_t)(c >> 6) * SLAB_BYTES + ((uint32_t)(((c >> 3) & 7) ^ (m & 7)) << 4);
                        float f[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) f[k] = valid ? __uint_as_float(v[g * 8 + k]) * scale : 0.f;
                        if (add_mode == 1 || gadd) {
                            const uint4 a0 = add_mode == 1 ? lds128(sa) : ga[g];
                            const uint32_t aw[4] = {a0.x, a0.y, a0.z, a0.w};
                            if (valid) {
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    f[2 * k] += __uint_as_float(aw[k] << 16);
                                    f[2 * k + 1] += __uint_as_float(aw[k] & 0xFFFF0000u);
                                }
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
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the bulk store reads what this thread wrote
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty + 8 * buf);     // this warp has read its quadrant of the accumulator
            bar_sync_epi(bid);                                   // the staging tile is complete
            if (dense && leader) {
                for (int j = 0; j < out_slabs; ++j) tma_store_2d(&pp->map_out, stg + (uint32_t)(j * SLAB_BYTES), col0 + j * 64, tm * TILE_M);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            if (stat_tiles) {
                // column sums of the stored (rounded) values: every warp over its own 32 rows, lane = two neighbouring columns;
                // the four warps' sums are then added in a fixed order
                for (int j = 0; j < out_slabs; ++j) {
                    float s0 = 0.f, s1 = 0.f, q0 = 0.f, q1 = 0.f;
#pragma unroll 8
                    for (int r = 0; r < 32; ++r) {
                        const int row = quad * 32 + r;
                        const uint32_t u = lds32(stg + (uint32_t)(j * SLAB_BYTES) + (uint32_t)row * 128u + ((uint32_t)((lane >> 2) ^ (row & 7)) << 4) + ((uint32_t)(lane & 3) << 2));
                        const float lo = __uint_as_float(u << 16), hi = __uint_as_float(u & 0xFFFF0000u);
                        s0 += lo; q0 += lo * lo; s1 += hi; q1 += hi * hi;
                    }
                    stat_s[quad][0][j * 64 + 2 * lane] = s0; stat_s[quad][0][j * 64 + 2 * lane + 1] = s1;
                    stat_s[quad][1][j * 64 + 2 * lane] = q0; stat_s[quad][1][j * 64 + 2 * lane + 1] = q1;
                }
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
            if (!dense) {
                // copy-out of a tall tile: 16-byte chunks, eight consecutive lanes per 128-byte run of one output pixel
                const int n_chunks = out_slabs * TILE_M * 8;
                for (int idx = et; idx < n_chunks; idx += 128) {
                    const int ch = idx & 7, row = (idx >> 3) & (TILE_M - 1), j = idx >> 10;
                    const int c = j * 64 + ch * 8, px = pix_s[row];
                    if (px >= 0 && c < n_tile && col0 + c < ncol)
                        *reinterpret_cast<uint4*>(outp + (long long)px * ncol + col0 + c) =
                            lds128(stg + (uint32_t)(j * SLAB_BYTES) + (uint32_t)row * 128u + ((uint32_t)(ch ^ (row & 7)) << 4));
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
    __shared__ __align__(8) uint64_t bars[2 * TC_MAX_STAGES + 1];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int shift8_s[4], wtap_s[4];                       // the group's taps: row shift in 16-byte units, index in dw
    const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[TC_MAX_STAGES]), bar_acc = smem_u32(&bars[2 * TC_MAX_STAGES]);
    const uint32_t ring = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
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
    } else if (warp == 1) {
        if (lane == 0) {
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
                for (int tt = 0; tt < ntap; ++tt) {
                    const uint32_t at16 = a16 + (uint32_t)shift8_s[tt];
                    const uint32_t d_t = tmem_d + (uint32_t)(tt * n_tile);
#pragma unroll
                    for (int k16 = 0; k16 < 8; ++k16)          // 16 positions = 16 rows of 128 bytes per step
                        umma_bf16(d_t, dy_const | (uint64_t)((dy16 + 128u * (uint32_t)k16) & 0x3FFFu), a_const | (uint64_t)((at16 + 128u * (uint32_t)k16) & 0x3FFFu), idesc, (i | k16) ? 1u : 0u);
                }
                umma_commit(bar_empty + 8 * s);
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(bar_acc);
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
                    if (nc > 0) { tmem_ld32(tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(tt * n_tile + c0), v);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
                    else { for (int j = 0; j < 32; ++j) v[j] = 0u; }
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
static bool tall_of(int Hg, int Wg, int pad, int es, Tall& t) {
    t.Wp = Wg + pad;
    const int H0 = Hg + pad;
    if (t.Wp * es > 256) return false;
    int best_r = 1, best_hp = H0;
    for (int r = 1; r <= H0; ++r) {
        const int hp = (H0 + r - 1) / r * r;
        if (r * t.Wp > 96 || r * es > 256 || (hp - H0) * 200 > 13 * H0 || (pad == 0 && hp != H0)) continue;   // pad = 0: positions are the pixels in order, no extra rows
        if (r * t.Wp > best_r * t.Wp) { best_r = r; best_hp = hp; }
    }
    t.Hp = best_hp; t.R = best_r; t.box_h = best_r; t.box_n = 1;
    if (best_r == best_hp) {                      // whole images: several per box when they are small
        int ni = 96 / (t.Hp * t.Wp); if (ni < 1) ni = 1; if (ni > 8) ni = 8;
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
        t.add_mode = !p.add ? 0 : p.add_sub == 2 ? 3 : t.dense ? 1 : 2;
        // output tiles: up to 256 columns (128 with a prefetched residual: several staging tiles), a multiple of 64 when there are several
        const int n_cap = t.add_mode == 1 ? 128 : 256;
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
            if (t.add_mode == 1 && !encode_flat(&tp.map_add, p.add, ncol, out_pixels)) return 0;
        }
        memcpy((char*)host_tc + (size_t)ph * sizeof(TcProb), &tp, sizeof(tp));
    }
    return count;
}
size_t conv_tc_prob_bytes() { return sizeof(TcProb); }
int conv_tc_tiles(const void* host_tc) { const TcHot* t = &((const TcProb*)host_tc)->h; return t->tiles_m * t->tiles_n; }
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
    L.prefetch = ((packed >> 36) & 0xF) > 1 ? 1 : 0;
    const size_t b_total = ((packed >> 20) & 0xFFFF) * 1024;
    const int n_tile = (int)(packed & 0xFFFFF);
    L.stg_bytes = ((n_tile + 63) / 64) * SLAB_BYTES;
    // Shared memory.  Staging tiles: two epilogue groups where they fit (they take alternate tiles, so two epilogues run side by
    // side), each with two tiles when the residual is prefetched into them by TMA, else one; a single group (three tiles behind a
    // prefetched residual) otherwise.  Weights: resident when all tiles of a column tile are small, else a ring of three tiles.  The
    // rest goes to the ring of activation windows: an HBM-bound layer runs at the bytes it keeps in flight.
    L.b_res = b_total <= TC_RESIDENT_BUDGET ? 1 : 0;
    const size_t kgroups = L.b_stage ? b_total / (size_t)L.b_stage : 1;
    const size_t b_min = L.b_res ? b_total : 2 * (size_t)L.b_stage;
    L.groups = 2; L.pg = L.prefetch ? 2 : 1;
    if (kgroups > 8) L.groups = 1;                             // long reductions: the epilogue is a small share, the smem goes to the rings
    if (L.groups == 1 || (size_t)L.groups * L.pg * L.stg_bytes + 3 * (size_t)L.a_stage + b_min > TC_SMEM_BUDGET) {
        L.groups = 1; L.pg = L.prefetch ? 3 : 1;
        while (L.pg > (L.prefetch ? 2 : 1) && (size_t)L.pg * L.stg_bytes + 2 * (size_t)L.a_stage + b_min > TC_SMEM_BUDGET) --L.pg;
    }
    L.n_stg = L.groups * L.pg;
    const size_t rings = TC_SMEM_BUDGET - (size_t)L.n_stg * L.stg_bytes;
    if (L.b_res) {
        L.nb = 0; L.b_region = (int)b_total;
        L.na = 2; while (L.na < TC_MAX_STAGES && (size_t)(L.na + 1) * L.a_stage + b_total <= rings) ++L.na;
    } else {
        L.nb = 3; while (L.nb > 2 && (size_t)L.nb * L.b_stage + 2 * (size_t)L.a_stage > rings) --L.nb;
        L.na = 2; while (L.na < TC_MAX_STAGES && (size_t)(L.na + 1) * L.a_stage + (size_t)L.nb * L.b_stage <= rings) ++L.na;
        while (L.nb < 6 && (size_t)L.na * L.a_stage + (size_t)(L.nb + 1) * L.b_stage <= rings) ++L.nb;
        L.b_region = L.nb * L.b_stage;
    }
    L.acc_stride = (n_tile + 31) / 32 * 32;
    L.tmem_cols = 32; while (L.tmem_cols < 2 * L.acc_stride) L.tmem_cols *= 2;
    // at least 120 KB of shared memory so that two CTAs that allocate tensor memory never share an SM
    const size_t smem = std::max((size_t)L.na * L.a_stage + (size_t)L.b_region + (size_t)L.n_stg * L.stg_bytes, (size_t)120 * 1024) + 1024;
    const long long total = (long long)max_tiles * nprob;
    const int grid = (int)std::max(1ll, std::min(total, (long long)sms));
    conv_tc_kernel<<<grid, TC_CONV_THREADS, smem, s>>>((const TcProb*)d_tc, L);
}

// ---- wgrad host side
struct WgGeom { TcWgradProb t; size_t smem, partial_bytes; int box_h, box_n; };

static bool wg_geometry(const ConvProb& p, int target_ctas, WgGeom& w) {
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
        Tall g; if (!tall_of(p.H, p.W, 1, 1, g)) return false;
        w.box_h = g.box_h; w.box_n = g.box_n;
        t.dy_flat = 0; t.a_flat = 0; t.pad = 1; t.Hp = g.Hp; t.Wp = g.Wp; t.R = g.R; t.box_pos = g.box_pos; t.hb = g.Wp + 1;
        t.nbox_dy = boxes_for(TILE_M, g.box_pos); t.nbox_a = boxes_for(TILE_M + 2 * t.hb, g.box_pos); t.dy_box_bytes = g.box_bytes; t.a_box_bytes = g.box_bytes;
        total_pos = (long long)p.N * g.Hp * g.Wp;
        for (int i = 0; i < 9; ++i) t.tap[i] = TapRef{i, (i / 3) * g.Wp + (i % 3)};
        t.tap_groups = 0;                                // groups of up to three taps: set below, once the column tile is known
    } else {
        Tall g; if (!tall_of(p.P, p.Q, 1, 2, g)) return false;
        Tall gd; if (!tall_of(p.P, p.Q, 1, 1, gd)) return false;
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
    t.tmem_cols = 32; while (t.tmem_cols < max_group * t.n_tile) t.tmem_cols *= 2;
    if (t.tmem_cols > 512) return false;
    t.dy_slab_bytes = (t.nbox_dy * t.dy_box_bytes + 1023) / 1024 * 1024;
    t.a_slab_bytes = (t.nbox_a * t.a_box_bytes + 1023) / 1024 * 1024;
    t.stage_bytes = 2 * t.dy_slab_bytes + t.a_slabs * t.a_slab_bytes;
    t.stages = TC_MAX_STAGES; while (t.stages > 1 && (size_t)t.stages * t.stage_bytes > TC_SMEM_BUDGET) --t.stages;
    if ((size_t)t.stages * t.stage_bytes > TC_SMEM_BUDGET) return false;
    w.smem = std::max((size_t)t.stages * t.stage_bytes, (size_t)120 * 1024) + 1024;
    const int fixed = t.m_tiles * t.n_tiles * t.tap_groups;
    int want = std::max(1, target_ctas / fixed); if (want > t.chunks) want = t.chunks; if (want > 256) want = 256;
    t.chunks_per_split = (t.chunks + want - 1) / want; t.splits = (t.chunks + t.chunks_per_split - 1) / t.chunks_per_split;
    w.partial_bytes = t.splits > 1 ? (size_t)t.splits * taps * p.K * p.C * 4 : 0;
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
