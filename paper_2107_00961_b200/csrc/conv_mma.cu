// Convolutions of NARROW layers (C and K multiples of 16, at most 64) on warp-level MMA (mma.sync m16n8k16, bf16
// inputs, fp32 accumulation).
//
// Why not tcgen05 here: one thread issues a tcgen05.mma (M = 128, K = 16) only every 114-165 cycles whatever its N, two
// issuing warps every 57-82 (resist_micro_mma_rate in micro.cu measures it), while the tensor core needs N / 2 cycles: a layer
// with 16 or 32 output channels would spend 4-10 times its tensor time on issue, and its TMA rows would be 32-64 bytes.  The
// warp-level MMA has no such granularity (n = 8), cp.async has no per-row cost, and these HBM-bound layers need far less
// than its rate.  Wider layers, and 64-channel 3x3 layers with many positions, run on tcgen05 (conv_tc.cu).
//
// Tiling: a GROUP of G whole images is one tall zero-padded map.  With pad = k/2, image n occupies rows
// n*Hp .. n*Hp+H-1 (Hp = H + pad) of a map that is Wp = W + pad wide; row H of every image and column W of every
// row are zero and serve as the padding of both neighbours, because positions are numbered row-major
// ("padded-flat", f = Y*Wp + X) and a tap (r, s) reads position f + (r-pad)*Wp + (s-pad).  A group is cut into
// pieces of SUB consecutive positions; the window a piece needs (piece + halo of pad*Wp + pad on either side) is
// staged in shared memory as [position][channel] rows, padded by 16 bytes against bank conflicts, and the k*k
// taps read it at shifted row offsets through ldmatrix.  Because a group starts on an image boundary, two small
// tables built once per CTA (window row -> input pixel, position -> output pixel; -1 at padding) serve every
// piece of every group: neither the copies nor the epilogue do any index arithmetic.
//
// Fused BatchNorm (bn.fuse != 0): at this problem size a layer is a few microseconds of work and a training step is a
// chain of dependent launches, so the BN+ReLU that consumes a convolution's output runs in the SAME launch.  The
// epilogue adds up the per-channel sums the BN needs (forward: x, x^2 of the stored bf16 output; backward: dz, dz*xhat
// with dz = da * [relu input > 0]) per CTA in a fixed order, the CTAs meet at a grid-wide barrier (cooperative launch),
// every CTA adds the per-CTA partial sums of its problem in the same fixed order, and the grid makes the elementwise
// pass over the tensor it has just written (an L2 hit).
#include <algorithm>
#include <cstring>
#include <cooperative_groups.h>
#include "internal.h"

namespace cg = cooperative_groups;

namespace resist {

struct alignas(16) MmaProb {
    const __nv_bfloat16* act;   // forward: a [n_img,H,W,ca]; dgrad: dy (stride 1, possibly zero-stuffed)
    const __nv_bfloat16* wgt;   // [K][taps][C]
    const __nv_bfloat16* add; __nv_bfloat16* out;
    int ca, ncol;               // channels of act (reduction) and of out
    int wC;                     // C of the weight tensor (its innermost extent)
    int H, W, Hp, Wp;           // image extent; extent of one image in the tall padded map
    unsigned inv_wp, inv_hp;    // floor(2^32 / d) + 1: __umulhi(f, inv) = f / d for every f the kernel meets
    int G, gpos;                // images per group, positions per group (G * Hp * Wp)
    int sub, subs, units;       // positions per piece (multiple of 16), pieces per group, pieces in total
    int os, P, Q;               // output stride (forward of a stride-2 layer stores even positions only, as a P x Q image)
    int is, iP, iQ;             // input stride: 2 = act is stored compact [n_img,iP,iQ,ca] and read as if zero-stuffed to H x W
    int stages;                 // depth of the activation ring (2, 3 or 4)
    int nsplit;                 // 1, or 2: a CTA computes one half of the output channels (its half of the filter resident)
    int variant, smem_bytes;    // which instantiation runs this problem (see mma_variant); dynamic shared memory
    float scale;
    int fuse;                   // 0: convolution only; 1: + BN+ReLU forward of out; 2: + BN+ReLU backward with out as da
    BnProb bn;                  // fuse 1: x = out, a; fuse 2: x, da = out, dx, add.  partial: [CTAs of the problem][2][C] doubles
};

__device__ __forceinline__ void bf8_unpack(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
}
__device__ __forceinline__ uint4 bf8_pack(const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]); w[i] = *reinterpret_cast<uint32_t*>(&h); }
    return make_uint4(w[0], w[1], w[2], w[3]);
}


__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t addr, uint32_t& r0, uint32_t& r1) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2_t(uint32_t addr, uint32_t& r0, uint32_t& r1) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int MMA_THREADS = 256;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");   // src_bytes 0: zeros
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// Programmatic dependent launch: a kernel launched with the attribute may start while the kernel before it in the
// stream is still running; it must not touch anything that kernel writes before pdl_wait() returns (which is when that
// kernel has finished and its writes are visible).  pdl_trigger() lets the NEXT kernel of the stream start early.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <class K, class A>
static void launch_pdl(K kernel, dim3 grid, size_t smem, cudaStream_t s, bool pdl, A arg) {
    cudaLaunchConfig_t cfg = {}; cfg.gridDim = grid; cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1]; at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization; at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = pdl ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, arg);
}
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Column n of the MMA's B operand carries output channel chan_of_col(n): thread (g8, t4) of a warp then owns, over its
// NB accumulator blocks, the 2*NB CONSECUTIVE channels t4*2*NB ... and stores them with 8- or 16-byte accesses.
template <int NB> __host__ __device__ __forceinline__ int chan_of_col(int n) { return ((n & 7) >> 1) * (2 * NB) + 2 * (n >> 3) + (n & 1); }
template <int NB> __host__ __device__ __forceinline__ int col_of_chan(int c) { return 8 * ((c % (2 * NB)) >> 1) + 2 * (c / (2 * NB)) + (c & 1); }


// Persistent: a CTA keeps the whole filter in shared memory and walks the pieces blockIdx.x, blockIdx.x + gridDim.x,
// ... of its problem.  The windows of the next pieces are in flight (cp.async, ring of p.stages) while the warps run
// ldmatrix + mma.sync on the current one.  Warp w computes the 16-row blocks w, w + 8, ... of a piece.
// NB = output channels / 8 (2, 4, 6 or 8); MBW = 16-row blocks per warp (a piece has at most 128 * MBW positions);
// KSZ = 1 or 3; TRANS = false: forward (weights read as [n][k]); true: dgrad (weights read as [k][n] and transposed
// on load, taps flipped).  CA = channels of the staged activations when the instance is specialised on them (all pitches
// and the reduction loop are then compile-time), 0 = read from the problem.
template <int NB, int MBW, int KSZ, bool TRANS, int CA>
__global__ void __launch_bounds__(MMA_THREADS, (NB == 2 && CA != 0) ? 3 : 2) conv_mma_kernel(   // registers for three (16-channel CTAs) or two CTAs per SM
const MmaProb* __restrict__ probs) {
    __shared__ MmaProb p;
    if (threadIdx.x < sizeof(MmaProb) / 4) reinterpret_cast<uint32_t*>(&p)[threadIdx.x] = reinterpret_cast<const uint32_t*>(probs + blockIdx.y)[threadIdx.x];
    __syncthreads();
    pdl_trigger();
    constexpr int TAPS = KSZ * KSZ, PAD = KSZ / 2, ncol = NB * 8;   // ncol: output channels of THIS CTA
    const int units = p.units, nsplit = p.nsplit;
    const int ncol_all = ncol * nsplit, n_off = ((int)blockIdx.x % nsplit) * ncol;
    const int cta = blockIdx.x / nsplit, ncta = gridDim.x / nsplit;   // the launcher makes gridDim.x a multiple of nsplit
    constexpr bool FUSABLE = NB <= 4;                             // wider CTAs would pay for the sums with registers: the host never asks
    const int fuse = FUSABLE ? p.fuse : 0;
    if (cta >= units && !fuse) return;                            // fused: every CTA must reach the grid barrier
    extern __shared__ __align__(16) uint8_t sm[];
    __shared__ float s_red[8][2][NB * 8];                         // per-warp sums of the fused BN, over the CTA's whole walk
    __shared__ float s_bn[4][NB * 8];                             // fuse 2: mean, 1/std, gamma, beta of this CTA's channels
    const int ca = CA ? CA : p.ca, apitch = ca * 2 + 16;          // activation row pitch in bytes
    const int wrows = TRANS ? ca : ncol;                          // rows of one tap of the staged filter
    const int wcols = TRANS ? ncol : ca;                          // elements per row
    const int wpitch = wcols * 2 + 16;
    const int Wp = p.Wp, sub = p.sub, subs = p.subs, stages = p.stages;
    const int halo = PAD * Wp + PAD, win_rows = sub + 2 * halo, nblk = sub / 16;
    const int it_rows = subs * sub + 2 * halo, ot_rows = subs * sub;
    short* itable = reinterpret_cast<short*>(sm);               // a group has fewer than 32768 pixels
    short* otable = itable + it_rows;
    const int table_bytes = ((it_rows + ot_rows) * 2 + 127) & ~127;
    const int stage_bytes = (win_rows * apitch + 127) & ~127;
    uint8_t* ring = sm + table_bytes;
    uint8_t* s_w = ring + stages * stage_bytes;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const __nv_bfloat16* __restrict__ act = p.act;
    const __nv_bfloat16* __restrict__ addp = p.add;
    __nv_bfloat16* __restrict__ outp = p.out;

    // ---- tables: window row w of a group (position f = w - halo) -> input pixel inside the group; position -> output pixel
    for (int w = tid; w < it_rows; w += MMA_THREADS) {
        const int f = w - halo;
        int pix = -1, opix = -1;
        if (f >= 0 && f < p.gpos) {
            const unsigned Y = __umulhi((unsigned)f, p.inv_wp), X = (unsigned)f - Y * Wp;
            const unsigned n = __umulhi(Y, p.inv_hp), i = Y - n * p.Hp;
            if (X < (unsigned)p.W && i < (unsigned)p.H) {
                if (p.is == 2) pix = ((i | X) & 1u) ? -1 : (int)((n * p.iP + (i >> 1)) * p.iQ + (X >> 1));   // zero-stuffed: only even positions exist
                else pix = (int)((n * p.H + i) * p.W + X);
                if (p.os == 1) opix = (int)((n * p.H + i) * p.W + X);
                else if (!((i % p.os) | (X % p.os))) opix = (int)((n * p.P + i / p.os) * p.Q + X / p.os);
            }
        }
        itable[w] = (short)pix;
        if (f >= 0 && f < ot_rows) otable[f] = (short)opix;
    }
    // ---- the filter, once per CTA
    if (!TRANS) {               // tap t, column n, 8-channel group g  <-  w[chan_of_col(n)][t][g*8..]
        const int groups = ca / 8, n_chunks = TAPS * ncol * groups;
        for (int id0 = tid; id0 < n_chunks; id0 += 4 * MMA_THREADS) {       // four loads in flight per thread
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int id = min(id0 + u * MMA_THREADS, n_chunks - 1);
                const int g = id % groups, n = (id / groups) % ncol, t = id / (groups * ncol);
                v[u] = __ldg(reinterpret_cast<const uint4*>(p.wgt + ((long long)(n_off + chan_of_col<NB>(n)) * TAPS + t) * p.wC + g * 8));
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int id = id0 + u * MMA_THREADS;
                if (id < n_chunks) { const int g = id % groups, n = (id / groups) % ncol, t = id / (groups * ncol);
                    *reinterpret_cast<uint4*>(s_w + (t * wrows + n) * wpitch + g * 16) = v[u]; }
            }
        }
    } else {                    // tap t, row k, column col_of_chan(c)  <-  w[k][t][c]
        constexpr int groups = ncol / 8; const int n_chunks = TAPS * ca * groups;
        for (int id0 = tid; id0 < n_chunks; id0 += 4 * MMA_THREADS) {       // four loads in flight per thread
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int id = min(id0 + u * MMA_THREADS, n_chunks - 1);
                const int g = id % groups, k = (id / groups) % ca, t = id / (groups * ca);
                v[u] = __ldg(reinterpret_cast<const uint4*>(p.wgt + ((long long)k * TAPS + t) * p.wC + n_off + g * 8));
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int id = id0 + u * MMA_THREADS;
                if (id < n_chunks) {
                    const int g = id % groups, k = (id / groups) % ca, t = id / (groups * ca);
                    const uint32_t w4[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                    uint8_t* row = s_w + (t * wrows + k) * wpitch;
#pragma unroll
                    for (int e = 0; e < 4; ++e) *reinterpret_cast<uint32_t*>(row + col_of_chan<NB>(g * 8 + 2 * e) * 2) = w4[e];   // channel pairs stay adjacent
                }
            }
        }
    }
    // ---- this thread's part of every copy: one 8-channel piece of every (256 / pieces-per-row)-th window row
    const int ga = ca / 8, a_step = MMA_THREADS / ga, a_row0 = tid / ga, a_g = tid % ga;
    const bool a_on = tid < a_step * ga;
    const long long grp_in = (long long)p.G * (p.is == 2 ? p.iP * p.iQ : p.H * p.W) * ca;   // elements of a group of act
    const long long grp_out = (long long)p.G * (p.os == 1 ? p.H * p.W : p.P * p.Q) * ncol_all;
    const __nv_bfloat16* pf_add = addp;
    const __nv_bfloat16* pf_x = fuse == 2 ? reinterpret_cast<const __nv_bfloat16*>(p.bn.x) : nullptr;
    auto issue = [&](int unit, int stage) {
        const int grp = unit / subs, j = unit - grp * subs;
        const __nv_bfloat16* ag = act + grp * grp_in + a_g * 8;
        if (a_on) {
            const short* t = itable + j * sub + a_row0;
            uint32_t dst = s_u32(ring + stage * stage_bytes) + a_g * 16 + a_row0 * apitch;
            for (int row = a_row0; row < win_rows; row += a_step, t += a_step, dst += a_step * apitch) {
                const int pix = *t;                                // padding: read nothing, write zeros
                cp_async16(dst, ag + (long long)max(pix, 0) * ca, pix >= 0 ? 16u : 0u);
            }
        }
        // what the epilogue of that piece will read besides its accumulators (the residual; the BN input of a fused
        // backward) was written long ago and is no longer in L2: ask for its 128-byte lines now
        if (pf_add != nullptr || pf_x != nullptr) {
            const short* ot = otable + j * sub;
            for (int r = tid; r < sub; r += MMA_THREADS) {
                const int op = ot[r];
                const long long e = grp * grp_out + (long long)op * ncol_all;
                if (op >= 0 && (e & 63) == 0) {
                    if (pf_add != nullptr) asm volatile("prefetch.global.L2 [%0];" ::"l"(pf_add + e));
                    if (pf_x != nullptr) asm volatile("prefetch.global.L2 [%0];" ::"l"(pf_x + e));
                }
            }
        }
    };

    const uint32_t w_base = s_u32(s_w);
    const int g8 = lane >> 2, t4 = lane & 3;
    // 16-row blocks of this warp; one past the piece repeats the last block (no branch in the inner loop) and is not stored
    uint32_t a_blk[MBW];
#pragma unroll
    for (int mb = 0; mb < MBW; ++mb) a_blk[mb] = (uint32_t)(min(warp + 8 * mb, nblk - 1) * 16 + (lane & 15)) * apitch + (lane >> 4) * 16;
    // B fragments of two 8-column blocks per ldmatrix.x4: lanes 0-7 / 8-15 address the two k halves of block j, lanes 16-31 those of block j+1
    const uint32_t b_lane = TRANS ? (uint32_t)(((lane >> 3) & 1) * 8 + (lane & 7)) * wpitch + (lane >> 4) * 16
                                  : (uint32_t)((lane >> 4) * 8 + (lane & 7)) * wpitch + ((lane >> 3) & 1) * 16;
    const float scale = p.scale;
    if (fuse) for (int i = tid; i < 8 * 2 * ncol; i += MMA_THREADS) (&s_red[0][0][0])[i] = 0.f;

    __syncthreads();                                              // tables complete
    pdl_wait();                                                   // from here on: tensors the previous kernel may have written
    const __nv_bfloat16* __restrict__ bnx = reinterpret_cast<const __nv_bfloat16*>(p.bn.x);
    if (fuse == 2 && tid < ncol) {
        const int c = n_off + tid;
        s_bn[0][tid] = p.bn.stat[c]; s_bn[1][tid] = p.bn.stat[p.bn.C + c]; s_bn[2][tid] = p.bn.gamma[c]; s_bn[3][tid] = p.bn.beta[c];
    }
    int nxt = cta;
    for (int st = 0; st < stages - 1; ++st) { if (nxt < units) issue(nxt, st); cp_async_commit(); nxt += ncta; }
    int stage = 0;
    for (int unit = cta; unit < units; unit += ncta) {
        { const int ps = stage == 0 ? stages - 1 : stage - 1; if (nxt < units) issue(nxt, ps); cp_async_commit(); nxt += ncta; }
        if (stages == 2) cp_async_wait<1>(); else if (stages == 3) cp_async_wait<2>(); else cp_async_wait<3>();
        __syncthreads();                                          // this piece's window (and, first time, the filter) is in shared memory

        const uint32_t a_base = s_u32(ring + stage * stage_bytes);
        float acc[MBW][NB][4];
#pragma unroll
        for (int mb = 0; mb < MBW; ++mb)
#pragma unroll
            for (int j = 0; j < NB; ++j) { acc[mb][j][0] = acc[mb][j][1] = acc[mb][j][2] = acc[mb][j][3] = 0.f; }
#pragma unroll
        for (int t = 0; t < TAPS; ++t) {
            constexpr int K1 = KSZ - 1;
            const int r = t / KSZ, q = t % KSZ;
            const int shift = TRANS ? ((K1 - r) * Wp + (K1 - q)) : (r * Wp + q);
            const uint32_t a_tap = a_base + (uint32_t)shift * apitch;
            const uint32_t w_tap = w_base + (uint32_t)(t * wrows) * wpitch + b_lane;
#pragma unroll
            for (int k0 = 0; k0 < ca; k0 += 16) {
                uint32_t a[MBW][4];
#pragma unroll
                for (int mb = 0; mb < MBW; ++mb) ldsm_x4(a_tap + a_blk[mb] + k0 * 2, a[mb][0], a[mb][1], a[mb][2], a[mb][3]);
#pragma unroll
                for (int j = 0; j < NB; j += 2) {
                    uint32_t b0, b1, b2, b3;
                    if (!TRANS) ldsm_x4(w_tap + (uint32_t)(j * 8) * wpitch + k0 * 2, b0, b1, b2, b3);
                    else ldsm_x4_t(w_tap + (uint32_t)k0 * wpitch + j * 16, b0, b1, b2, b3);
#pragma unroll
                    for (int mb = 0; mb < MBW; ++mb) {
                        mma16816(acc[mb][j], a[mb][0], a[mb][1], a[mb][2], a[mb][3], b0, b1);
                        mma16816(acc[mb][j + 1], a[mb][0], a[mb][1], a[mb][2], a[mb][3], b2, b3);
                    }
                }
            }
        }
        // ---- epilogue: thread (g8, t4) holds rows g8 and g8+8 of each 16-row block, channels t4*2*NB ... t4*2*NB + 2*NB - 1.
        // No branch around the loads: a row at a padding position reads pixel 0 and is neither stored nor counted, so the
        // loads of all rows can be in flight together.
        const int grp = unit / subs, j0 = (unit - grp * subs) * sub;
        const long long obase = grp * grp_out + n_off + t4 * (2 * NB);
        const __nv_bfloat16* __restrict__ add_g = addp + obase;
        const __nv_bfloat16* __restrict__ bnx_g = bnx + obase;
        __nv_bfloat16* __restrict__ out_g = outp + obase;
        int opx[MBW][2];
#pragma unroll
        for (int mb = 0; mb < MBW; ++mb) {
            const int blk = min(warp + 8 * mb, nblk - 1);
            const bool real = warp + 8 * mb < nblk;
#pragma unroll
            for (int half = 0; half < 2; ++half) { const int v = otable[j0 + blk * 16 + g8 + half * 8]; opx[mb][half] = real ? v : -1; }
        }
        float ps[2 * NB], pq[2 * NB];                             // fused BN: this thread's sums over the piece
#pragma unroll
        for (int i = 0; i < 2 * NB; ++i) { ps[i] = 0.f; pq[i] = 0.f; }
#pragma unroll
        for (int mb = 0; mb < MBW; ++mb)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int opix = opx[mb][half];
                const bool valid = opix >= 0;
                const int o = max(opix, 0) * ncol_all;            // a tensor of one problem has fewer than 2^31 elements
                uint32_t wv[NB], xv[NB];
                if (addp) {
                    if constexpr (NB % 4 == 0) {
#pragma unroll
                        for (int c4 = 0; c4 < NB / 4; ++c4) { const uint4 v = *reinterpret_cast<const uint4*>(add_g + o + c4 * 8); wv[c4 * 4] = v.x; wv[c4 * 4 + 1] = v.y; wv[c4 * 4 + 2] = v.z; wv[c4 * 4 + 3] = v.w; }
                    } else {
#pragma unroll
                        for (int c2 = 0; c2 < NB / 2; ++c2) { const uint2 v = *reinterpret_cast<const uint2*>(add_g + o + c2 * 4); wv[c2 * 2] = v.x; wv[c2 * 2 + 1] = v.y; }
                    }
                }
                if (fuse == 2) {
                    if constexpr (NB % 4 == 0) {
#pragma unroll
                        for (int c4 = 0; c4 < NB / 4; ++c4) { const uint4 v = *reinterpret_cast<const uint4*>(bnx_g + o + c4 * 8); xv[c4 * 4] = v.x; xv[c4 * 4 + 1] = v.y; xv[c4 * 4 + 2] = v.z; xv[c4 * 4 + 3] = v.w; }
                    } else {
#pragma unroll
                        for (int c2 = 0; c2 < NB / 2; ++c2) { const uint2 v = *reinterpret_cast<const uint2*>(bnx_g + o + c2 * 4); xv[c2 * 2] = v.x; xv[c2 * 2 + 1] = v.y; }
                    }
                }
#pragma unroll
                for (int j = 0; j < NB; ++j) {
                    float v0 = acc[mb][j][half * 2] * scale, v1 = acc[mb][j][half * 2 + 1] * scale;
                    if (addp) { v0 += __uint_as_float(wv[j] << 16); v1 += __uint_as_float(wv[j] & 0xFFFF0000u); }
                    __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
                    wv[j] = *reinterpret_cast<uint32_t*>(&h);
                }
                if (fuse == 1) {                                  // sums of the STORED values: x, x^2
#pragma unroll
                    for (int j = 0; j < NB; ++j) {
                        const float r0 = valid ? __uint_as_float(wv[j] << 16) : 0.f, r1 = valid ? __uint_as_float(wv[j] & 0xFFFF0000u) : 0.f;
                        ps[2 * j] += r0; pq[2 * j] += r0 * r0; ps[2 * j + 1] += r1; pq[2 * j + 1] += r1 * r1;
                    }
                } else if (fuse == 2) {                           // sums of dz = da * [relu input > 0] and dz * xhat
#pragma unroll
                    for (int j = 0; j < NB; ++j) {
                        const int c = t4 * (2 * NB) + 2 * j;
                        const float2 mean = *reinterpret_cast<const float2*>(&s_bn[0][c]), istd = *reinterpret_cast<const float2*>(&s_bn[1][c]);
                        const float2 ga = *reinterpret_cast<const float2*>(&s_bn[2][c]), be = *reinterpret_cast<const float2*>(&s_bn[3][c]);
                        const float xh0 = (__uint_as_float(xv[j] << 16) - mean.x) * istd.x, xh1 = (__uint_as_float(xv[j] & 0xFFFF0000u) - mean.y) * istd.y;
                        const float dz0 = (valid && xh0 * ga.x + be.x > 0.f) ? __uint_as_float(wv[j] << 16) : 0.f;
                        const float dz1 = (valid && xh1 * ga.y + be.y > 0.f) ? __uint_as_float(wv[j] & 0xFFFF0000u) : 0.f;
                        ps[2 * j] += dz0; pq[2 * j] += dz0 * xh0; ps[2 * j + 1] += dz1; pq[2 * j + 1] += dz1 * xh1;
                    }
                }
                if (valid) {
                    if constexpr (NB % 4 == 0) {
#pragma unroll
                        for (int c4 = 0; c4 < NB / 4; ++c4) *reinterpret_cast<uint4*>(out_g + o + c4 * 8) = make_uint4(wv[c4 * 4], wv[c4 * 4 + 1], wv[c4 * 4 + 2], wv[c4 * 4 + 3]);
                    } else {
#pragma unroll
                        for (int c2 = 0; c2 < NB / 2; ++c2) *reinterpret_cast<uint2*>(out_g + o + c2 * 4) = make_uint2(wv[c2 * 2], wv[c2 * 2 + 1]);
                    }
                }
            }
        if (fuse) {                                               // the 8 lanes that own the same channels, fixed butterfly; lane g8 = 0 keeps the warp's running sum
#pragma unroll
            for (int i = 0; i < 2 * NB; ++i) {
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) { ps[i] += __shfl_xor_sync(0xffffffffu, ps[i], off); pq[i] += __shfl_xor_sync(0xffffffffu, pq[i], off); }
            }
            if (g8 == 0) {
#pragma unroll
                for (int i = 0; i < 2 * NB; ++i) { s_red[warp][0][t4 * (2 * NB) + i] += ps[i]; s_red[warp][1][t4 * (2 * NB) + i] += pq[i]; }
            }
        }
        __syncthreads();                                          // every warp is done with this stage before it is refilled
        stage = stage + 1 == stages ? 0 : stage + 1;
    }
    cp_async_wait<0>();
    if (!fuse) return;

    // ---- fused BN: this CTA's sums (warps added in order, in double) -> partial[cta][2][C]; grid barrier; statistics; elementwise pass
    const BnProb& bn = p.bn;
    const int C = bn.C;                                           // = ncol_all
    __syncthreads();
    if (cta < units && tid < 2 * ncol) {
        const int k = tid / ncol, c = tid - k * ncol;
        double a = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) a += (double)s_red[w][k][c];
        bn.partial[((long long)cta * 2 + k) * C + n_off + c] = a;
    }
    __threadfence();
    cg::this_grid().sync();
    float* s_stat = reinterpret_cast<float*>(sm);                 // [6][C]: mean, 1/std, sum dz, sum dz*xhat, gamma, beta (the tables are no longer needed)
    double* s_dred = reinterpret_cast<double*>(sm + 6 * 64 * 4);  // [2][256]
    {
        const int rows = min(ncta, units), Q = MMA_THREADS / C, c = tid % C, q = tid / C;   // C is 16, 32 or 64
        double a0 = 0.0, a1 = 0.0;
        {   // 8 rows (16 loads) in flight per thread: the loop is bound by L2 latency, not by its few kilobytes
            const double* pp = bn.partial + (long long)q * 2 * C + c;
            const long long step = (long long)Q * 2 * C;
            int k = q;
            for (; k + 7 * Q < rows; k += 8 * Q, pp += 8 * step) {
                double v0[8], v1[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) { v0[u] = __ldcg(pp + u * step); v1[u] = __ldcg(pp + u * step + C); }
#pragma unroll
                for (int u = 0; u < 8; ++u) { a0 += v0[u]; a1 += v1[u]; }
            }
            for (; k < rows; k += Q, pp += step) { a0 += __ldcg(pp); a1 += __ldcg(pp + C); }
        }
        s_dred[tid] = a0; s_dred[256 + tid] = a1;
        __syncthreads();
        if (q == 0) {
            a0 = 0.0; a1 = 0.0;
            for (int k = 0; k < Q; ++k) { a0 += s_dred[k * C + c]; a1 += s_dred[256 + k * C + c]; }
            if (fuse == 1) {
                const double m = (double)bn.m, mean = a0 / m;
                double var = a1 / m - mean * mean; if (var < 0.0) var = 0.0;
                const float fm = (float)mean, fi = (float)(1.0 / sqrt(var + (double)bn.eps));
                s_stat[c] = fm; s_stat[C + c] = fi;
                if (blockIdx.x == 0) {
                    bn.stat[c] = fm; bn.stat[C + c] = fi;
                    if (bn.run_mean) {
                        const double unb = bn.m > 1 ? var * m / (m - 1.0) : var, mo = (double)bn.momentum;
                        bn.run_mean[c] = (float)((1.0 - mo) * (double)bn.run_mean[c] + mo * mean);
                        bn.run_var[c] = (float)((1.0 - mo) * (double)bn.run_var[c] + mo * unb);
                    }
                }
            } else {
                s_stat[c] = bn.stat[c]; s_stat[C + c] = bn.stat[C + c];
                s_stat[2 * C + c] = (float)a0; s_stat[3 * C + c] = (float)a1;
                if (blockIdx.x == 0) { bn.stat[2 * C + c] = (float)a0; bn.stat[3 * C + c] = (float)a1; bn.dbeta[c] = (float)a0; bn.dgamma[c] = (float)a1; }
            }
        }
        __syncthreads();
    }
    // elementwise pass, 8 channels per access; the per-channel constants are read from shared memory where they are used
    // (kept in registers they would raise the register count of the whole kernel)
    {
        if (tid < C) { s_stat[4 * C + tid] = bn.gamma[tid]; s_stat[5 * C + tid] = bn.beta[tid]; }
        __syncthreads();
        const int G = C >> 3;
        const long long nv = bn.m * G, stride = (long long)gridDim.x * MMA_THREADS;
        const float inv_m = 1.f / (float)bn.m;
        const uint4* xv = reinterpret_cast<const uint4*>(bn.x);
        const uint4* dv = reinterpret_cast<const uint4*>(bn.da);
        const uint4* av = reinterpret_cast<const uint4*>(bn.add);
        uint4* ov = reinterpret_cast<uint4*>(fuse == 1 ? bn.a : bn.dx);
        for (long long v = (long long)blockIdx.x * MMA_THREADS + tid; v < nv; v += stride) {
            const float* st = s_stat + ((int)v & (G - 1)) * 8;
            float x[8], o[8]; bf8_unpack(__ldcg(xv + v), x);
            if (fuse == 1) {
#pragma unroll
                for (int j = 0; j < 8; ++j) { const float z = (x[j] - st[j]) * st[C + j] * st[4 * C + j] + st[5 * C + j]; o[j] = z > 0.f ? z : 0.f; }
            } else {
                float d[8]; bf8_unpack(__ldcg(dv + v), d);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float istd = st[C + j], ga = st[4 * C + j];
                    const float xh = (x[j] - st[j]) * istd;
                    const float dz = (xh * ga + st[5 * C + j] > 0.f) ? d[j] : 0.f;
                    o[j] = ga * istd * (dz - st[2 * C + j] * inv_m - xh * st[3 * C + j] * inv_m);
                }
                if (av) { float ad[8]; bf8_unpack(__ldcg(av + v), ad);
#pragma unroll
                    for (int j = 0; j < 8; ++j) o[j] += ad[j]; }
            }
            ov[v] = bf8_pack(o);
        }
    }
}

// ------------------------------------------------------------------------------------------------ host side
struct MmaGeom { int ca, ncol, Hp, Wp, G, gpos, sub, subs, units, mbw, stages, nsplit, variant; size_t smem; };

// variant = ((MBW * 4 + ksz) * 2 + trans) * 16 + NB: everything a launch is specialised on; + MMA_VARIANT_FUSED: with BN
constexpr int MMA_VARIANT_FUSED = 512;
// + (1, 2, 3) << 10: a 3x3 instance specialised on 16, 32 or 64 staged channels (CTAs of 16 or 32 output channels)
static int mma_ca_code(int ksz, int nb, int ca) { return ksz == 3 && (nb == 2 || nb == 4) ? (ca == 16 ? 1 : ca == 32 ? 2 : ca == 64 ? 3 : 0) : 0; }
static int mma_variant(int mbw, int ksz, int trans, int nb) { return ((mbw * 4 + ksz) * 2 + trans) * 16 + nb; }

static bool mma_geometry(const ConvProb& p, int mode, MmaGeom& g) {
    if (mode == CONV_WGRAD) return false;
    if ((p.ksz != 1 && p.ksz != 3) || p.stride < 1 || p.stride > 2 || (p.stride == 2 && mode != CONV_FWD)) return false;
    if (p.C % 16 || p.K % 16 || p.C > 64 || p.K > 64 || p.N < 1) return false;
    if (((uintptr_t)p.act | (uintptr_t)p.wgt | (uintptr_t)p.out | (uintptr_t)p.add) & 15) return false;
    g.ca = mode == CONV_FWD ? p.C : p.K; g.ncol = mode == CONV_FWD ? p.K : p.C;
    const int pad = p.ksz / 2;
    g.Hp = p.H + pad; g.Wp = p.W + pad;
    if (g.Hp < 2 || g.Wp < 2) return false;
    const int ppi = g.Hp * g.Wp, halo = pad * g.Wp + pad;
    const int apitch = g.ca * 2 + 16;
    const int wrows = mode == CONV_FWD ? g.ncol : g.ca, wcols = mode == CONV_FWD ? g.ca : g.ncol;
    // 64 output channels: two CTAs share a piece, each with half of the filter resident (twice the CTAs per SM).  (A split
    // in four on the 8x8 stage, with three 16-channel CTAs per SM, was measured: no faster, the window is staged four times.)
    g.nsplit = g.ncol == 64 && p.ksz == 3 ? 2 : 1;
    const int ncta_col = g.ncol / g.nsplit;
    const int wrows_c = mode == CONV_FWD ? ncta_col : g.ca, wcols_c = mode == CONV_FWD ? g.ca : ncta_col;
    const size_t wbytes = (size_t)p.ksz * p.ksz * wrows_c * (wcols_c * 2 + 16);
    (void)wrows; (void)wcols;
    const int max_mbw = ncta_col <= 32 ? 3 : 2;                   // accumulators: MBW * (channels / 8) * 4 registers
    // images per group and positions per piece: little padding of the last piece, all warps busy, pieces not too
    // small, enough pieces to go round
    double best = 1e30; g.sub = 0;
    for (int G = 1; G <= std::min(p.N, 64); ++G) {
        if (p.N % G) continue;
        const int gpos = G * ppi;
        if (gpos > 3000 && g.sub) break;
        if (gpos > 7000) break;
        for (int sub = 64; sub <= 128 * max_mbw; sub += 16) {
            const int subs = (gpos + sub - 1) / sub, nblk = sub / 16, mbw = (nblk + 7) / 8;
            if (gpos >= 32768 || (long long)G * p.H * p.W >= 32768) continue;
            const size_t table = (size_t)(((2 * subs * sub + 2 * halo) * 2 + 127) & ~127);
            const size_t stage = (size_t)(((sub + 2 * halo) * apitch + 127) & ~127);
            // 16-channel CTAs need few registers: three of them share an SM when each stays below 72 KB
            const size_t budget = (ncta_col <= 16 && table + 2 * stage + wbytes + 64 <= 72 * 1024) ? 72 * 1024 : 100 * 1024;
            int stages = 4; while (stages > 2 && table + stages * stage + wbytes + 64 > budget) --stages;
            if (table + stages * stage + wbytes + 64 > 200 * 1024) continue;
            const long long units = (long long)(p.N / G) * subs;
            double cost = (double)subs * sub / gpos * (1.0 + 48.0 / sub) * (8.0 * mbw / nblk);
            if (units < 64) cost *= 1.0 + 0.5 * (64 - units) / 64.0;
            if (cost < best) { best = cost; g.G = G; g.gpos = gpos; g.sub = sub; g.subs = subs; g.units = (int)units; g.mbw = mbw; g.stages = stages;
                               g.smem = table + stages * stage + wbytes + 64; }
        }
    }
    if (!g.sub) return false;
    g.variant = mma_variant(g.mbw, p.ksz, mode == CONV_DGRAD ? 1 : 0, ncta_col / 8) | (mma_ca_code(p.ksz, ncta_col / 8, g.ca) << 10);
    return true;
}

bool conv_mma_supported(const ConvProb& p, int mode) { MmaGeom g; return mma_geometry(p, mode, g); }
int conv_mma_pick_variant(const ConvProb& p, int mode) { MmaGeom g; return mma_geometry(p, mode, g) ? g.variant : 0; }
size_t conv_mma_prob_bytes() { return sizeof(MmaProb); }

// bn != nullptr: the BN+ReLU that consumes the output runs in the same launch (forward of mode CONV_FWD, backward of
// CONV_DGRAD); bn->partial must hold conv_mma_bn_partial_bytes(C) bytes
size_t conv_mma_bn_partial_bytes(int C, int sms) { return (size_t)3 * sms * 2 * C * sizeof(double); }
bool conv_mma_can_fuse_bn(const ConvProb& p, int mode, int C) {
    MmaGeom g; if (!mma_geometry(p, mode, g)) return false;
    return (C == 16 || C == 32 || C == 64) && C == g.ncol && g.ncol / g.nsplit <= 32;
}
bool conv_mma_fill(const ConvProb& p, int mode, void* host, const BnProb* bn) {
    MmaGeom g; if (!mma_geometry(p, mode, g)) return false;
    MmaProb t; memset(&t, 0, sizeof(t));
    t.act = (const __nv_bfloat16*)p.act; t.wgt = (const __nv_bfloat16*)p.wgt; t.add = (const __nv_bfloat16*)p.add; t.out = (__nv_bfloat16*)p.out;
    t.ca = g.ca; t.ncol = g.ncol; t.wC = p.C; t.H = p.H; t.W = p.W; t.Hp = g.Hp; t.Wp = g.Wp;
    t.inv_wp = (unsigned)((1ull << 32) / (unsigned)g.Wp + 1); t.inv_hp = (unsigned)((1ull << 32) / (unsigned)g.Hp + 1);
    t.G = g.G; t.gpos = g.gpos; t.sub = g.sub; t.subs = g.subs; t.units = g.units;
    t.os = mode == CONV_FWD ? p.stride : 1; t.P = p.P; t.Q = p.Q;
    t.is = (mode == CONV_DGRAD && p.dy_sub == 2) ? 2 : 1; t.iP = p.dy_P; t.iQ = p.dy_Q;
    t.stages = g.stages; t.nsplit = g.nsplit; t.variant = g.variant; t.smem_bytes = (int)g.smem; t.scale = p.scale;
    if (bn) {
        if (!conv_mma_can_fuse_bn(p, mode, bn->C)) return false;
        t.fuse = mode == CONV_FWD ? 1 : 2; t.bn = *bn; t.variant |= MMA_VARIANT_FUSED;
        if (t.smem_bytes < 8192) t.smem_bytes = 8192;             // the BN phase reuses the start of the dynamic shared memory (5.5 KB)
    }
    memcpy(host, &t, sizeof(t));
    return true;
}
int conv_mma_tiles(const void* h) { return ((const MmaProb*)h)->units * ((const MmaProb*)h)->nsplit; }
int conv_mma_variant(const void* h) { return ((const MmaProb*)h)->variant; }
size_t conv_mma_smem(const void* h) { return (size_t)((const MmaProb*)h)->smem_bytes; }

struct MmaLaunch { const void* d; int nprob, max_tiles; size_t smem; bool pdl, coop; cudaStream_t s; bool ok; };

// Persistent CTAs: as many as are co-resident at this shared-memory footprint (at most 3 per SM), over all problems.
// A fused launch is cooperative (grid barrier): its grid never exceeds what is co-resident.
template <int NB, int MBW, int KSZ, bool TRANS, int CA = 0>
static void launch_mma_inst(MmaLaunch& a) {
    static bool configured = false; static int sms = 0; static signed char occ[256] = {};
    static int coop_pdl = 1;                                      // 1: cooperative + programmatic launch together until the driver refuses it
    auto kernel = conv_mma_kernel<NB, MBW, KSZ, TRANS, CA>;
    if (!configured) {
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 202 * 1024);
        int dev = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev); if (sms < 1) sms = 148;
        configured = true;
    }
    const int slot = (int)std::min<size_t>(a.smem / 1024, 255);
    if (!occ[slot]) { int n = 0; cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, MMA_THREADS, (a.smem / 1024 + 1) * 1024); occ[slot] = (signed char)std::max(1, std::min(n, 3)); }
    const int cap = occ[slot] * sms;
    int gx = a.coop ? cap / a.nprob : (cap + a.nprob - 1) / a.nprob;
    if (gx > a.max_tiles) gx = a.max_tiles;
    gx &= ~1;                                                     // even: a CTA pair shares a piece when the channels are split
    if (gx < 2) gx = 2;
    if (a.coop && gx * a.nprob > cap) { a.ok = false; return; }
    cudaLaunchConfig_t cfg = {}; cfg.gridDim = dim3(gx, a.nprob); cfg.blockDim = dim3(MMA_THREADS); cfg.dynamicSmemBytes = a.smem; cfg.stream = a.s;
    cudaLaunchAttribute at[2]; int n = 0;
    if (a.coop) { at[n].id = cudaLaunchAttributeCooperative; at[n].val.cooperative = 1; ++n; }
    if (a.pdl && (!a.coop || coop_pdl)) { at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization; at[n].val.programmaticStreamSerializationAllowed = 1; ++n; }
    cfg.attrs = at; cfg.numAttrs = n;
    const MmaProb* d = (const MmaProb*)a.d;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, d);
    if (e != cudaSuccess && a.coop && n == 2) {                   // the combination is refused: cooperative alone from now on
        cudaGetLastError(); coop_pdl = 0; cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kernel, d);
    }
    a.ok = e == cudaSuccess;
}
template <int NB, int MBW>
static void launch_mma_ca(MmaLaunch& a, int trans, int cac) {      // 3x3 instances specialised on the staged channels
    if (trans) { if (cac == 1) launch_mma_inst<NB, MBW, 3, true, 16>(a); else if (cac == 2) launch_mma_inst<NB, MBW, 3, true, 32>(a); else launch_mma_inst<NB, MBW, 3, true, 64>(a); }
    else { if (cac == 1) launch_mma_inst<NB, MBW, 3, false, 16>(a); else if (cac == 2) launch_mma_inst<NB, MBW, 3, false, 32>(a); else launch_mma_inst<NB, MBW, 3, false, 64>(a); }
}
template <int NB, int MBW>
static void launch_mma_nb(MmaLaunch& a, int ksz, int trans) {
    if (ksz == 3) { if (trans) launch_mma_inst<NB, MBW, 3, true>(a); else launch_mma_inst<NB, MBW, 3, false>(a); }
    else { if (trans) launch_mma_inst<NB, MBW, 1, true>(a); else launch_mma_inst<NB, MBW, 1, false>(a); }
}
// all problems of one launch share the variant
// pdl: the kernel may start before the previous kernel of the stream has finished (that kernel must not write the weights)
bool launch_conv_mma_probs(const void* d, int nprob, int max_tiles, size_t max_smem, int variant, cudaStream_t s, bool pdl) {
    const int nb = variant & 15, trans = (variant >> 4) & 1, ksz = (variant >> 5) & 3, mbw = (variant >> 7) & 3;
    MmaLaunch a{d, nprob, max_tiles, max_smem, pdl, (variant & MMA_VARIANT_FUSED) != 0, s, false};
    const int cac = (variant >> 10) & 3;
    if (cac && ksz == 3 && (nb == 2 || nb == 4) && mbw >= 1 && mbw <= 3) {
        if (nb == 2) { if (mbw == 1) launch_mma_ca<2, 1>(a, trans, cac); else if (mbw == 2) launch_mma_ca<2, 2>(a, trans, cac); else launch_mma_ca<2, 3>(a, trans, cac); }
        else { if (mbw == 1) launch_mma_ca<4, 1>(a, trans, cac); else if (mbw == 2) launch_mma_ca<4, 2>(a, trans, cac); else launch_mma_ca<4, 3>(a, trans, cac); }
        return a.ok;
    }
#define MMA_CASE(N_, M_) if (nb == N_ && mbw == M_) launch_mma_nb<N_, M_>(a, ksz, trans); else
    MMA_CASE(2, 1) MMA_CASE(2, 2) MMA_CASE(2, 3) MMA_CASE(4, 1) MMA_CASE(4, 2) MMA_CASE(4, 3)
    MMA_CASE(6, 1) MMA_CASE(6, 2) MMA_CASE(8, 1) MMA_CASE(8, 2)
    return false;
#undef MMA_CASE
    return a.ok;
}

// ------------------------------------------------------------------------------------------------ wgrad
// dw[k][t][c] = sum over positions f of dy[f][k] * a[f + shift_t][c], on the tall padded map of the forward kernel
// (dy and a read as zero at its padding positions).  GEMM with M = output channels, N = (tap, input channel) and
// the reduction over positions.
//
// Work is cut into GROUPS of G whole images (G * Hp * Wp positions) and each group into SUB-position pieces.  Because
// a group starts on an image boundary, one table (position in the group's window -> pixel index, or -1 at padding)
// built once per CTA serves every piece of every group: staging a piece is a table lookup and a cp.async per 16
// bytes, with no index arithmetic.  A CTA walks pieces blockIdx-strided with a ring of stages in flight; its 8
// warps form a WP x WN grid: a warp takes every WP-th 16-position step of a piece and, for ALL 16-row blocks of M,
// PPW pairs of 8-column blocks of N, and keeps those accumulators in registers over the whole walk.  At the end the
// WP partial sums are added in a fixed order through shared memory, the CTA writes one fp32 partial, and a second
// kernel adds the partials of all CTAs in a fixed order.
struct alignas(16) MmaWgradProb {
    const __nv_bfloat16* dy;    // [n_img,H,W,K]  (stride 1; a stride-2 layer passes the zero-stuffed dy)
    const __nv_bfloat16* a;     // [n_img,H,W,C]
    float* partial;             // [splits][taps][K][C]
    float* out;                 // [K][taps][C]
    int K, C, H, W, Hp, Wp, ksz, taps;
    int G, n_groups, gpos;      // images per group, groups, positions per group (G * Hp * Wp)
    int sub, subs, units;       // positions per piece (multiple of 16 * WP), pieces per group, pieces in total
    int table_rows;             // subs * sub + 2 * halo
    int tap_groups, taps_per_group, splits;
    int wn, stages, variant, smem_bytes;
    unsigned inv_wp, inv_hp;
    int out_ld, out_cols;       // 1x1 problems only: row stride and valid columns of out (an im2col'ed stem); else C, C
    int ds, dP, dQ;             // 2 = dy is stored compact [n_img,dP,dQ,K] and read as if zero-stuffed to H x W (a second table maps its rows)
};

template <int MB, int PPW>   // MB = K / 16; PPW = pairs of 8-column blocks a warp owns
__global__ void __launch_bounds__(MMA_THREADS) conv_wgrad_mma_kernel(const MmaWgradProb* __restrict__ probs) {
    __shared__ MmaWgradProb p;
    if (threadIdx.x < sizeof(MmaWgradProb) / 4) reinterpret_cast<uint32_t*>(&p)[threadIdx.x] = reinterpret_cast<const uint32_t*>(probs + blockIdx.y)[threadIdx.x];
    __syncthreads();
    pdl_trigger();
    if ((int)blockIdx.x >= p.tap_groups * p.splits) return;
    const int split = blockIdx.x % p.splits, tg = blockIdx.x / p.splits;
    const int tap0 = tg * p.taps_per_group; int ntap = p.taps - tap0; if (ntap > p.taps_per_group) ntap = p.taps_per_group;
    extern __shared__ __align__(16) uint8_t sm[];
    const int K = p.K, C = p.C, dpitch = K * 2 + 16, apitch = C * 2 + 16, Wp = p.Wp, sub = p.sub, subs = p.subs, stages = p.stages;
    const int pad = p.ksz / 2, halo = pad * Wp + pad, rows_a = sub + 2 * halo;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int WN = p.wn, WP = 8 / WN, warp_n = warp % WN, warp_p = warp / WN;
    int* table = reinterpret_cast<int*>(sm);
    const int table_bytes = (p.table_rows * 4 + 127) & ~127;
    const int dy_bytes = (sub * dpitch + 127) & ~127, stage_bytes = dy_bytes + ((rows_a * apitch + 127) & ~127);
    uint8_t* ring = sm + table_bytes;

    // ---- window row w of a group (position f = w - halo of the group) -> pixel index inside the group, -1 at padding
    for (int w = tid; w < p.table_rows; w += MMA_THREADS) {
        const int f = w - halo;
        int pix = -1;
        if (f >= 0 && f < p.gpos) {
            const unsigned Y = __umulhi((unsigned)f, p.inv_wp), X = (unsigned)f - Y * Wp;
            const unsigned n = __umulhi(Y, p.inv_hp), i = Y - n * p.Hp;
            if (X < (unsigned)p.W && i < (unsigned)p.H) pix = (int)((n * p.H + i) * p.W + X);
        }
        table[w] = pix;
    }
    // zero-stuffed dy: position f of a group -> pixel of the compact dy (even positions), -1 elsewhere
    const bool stuffed = p.ds == 2;
    int* dtable = reinterpret_cast<int*>(sm + table_bytes);
    const int dtable_bytes = stuffed ? ((subs * sub * 4 + 127) & ~127) : 0;
    if (stuffed) {
        for (int f = tid; f < subs * sub; f += MMA_THREADS) {
            int pix = -1;
            if (f < p.gpos) {
                const unsigned Y = __umulhi((unsigned)f, p.inv_wp), X = (unsigned)f - Y * Wp;
                const unsigned n = __umulhi(Y, p.inv_hp), i = Y - n * p.Hp;
                if (X < (unsigned)p.W && i < (unsigned)p.H && !((i | X) & 1u)) pix = (int)((n * p.dP + (i >> 1)) * p.dQ + (X >> 1));
            }
            dtable[f] = pix;
        }
    }
    ring += dtable_bytes;
    // ---- this thread's part of every copy: one 8-channel piece of every (256 / pieces-per-row)-th row
    const int ga = C / 8, gd = K / 8;
    const int a_step = MMA_THREADS / ga, d_step = MMA_THREADS / gd;           // rows per sweep (threads past step * g idle)
    const int a_row0 = tid / ga, a_g = tid % ga, d_row0 = tid / gd, d_g = tid % gd;
    const bool a_on = tid < a_step * ga, d_on = tid < d_step * gd;
    const long long img_a = (long long)p.H * p.W * C, img_d = (stuffed ? (long long)p.dP * p.dQ : (long long)p.H * p.W) * K;
    const __nv_bfloat16* __restrict__ a_ptr = p.a; const __nv_bfloat16* __restrict__ dy_ptr = p.dy;
    auto issue = [&](int unit, int stage) {
        const int grp = unit / subs, j = unit - grp * subs;
        const __nv_bfloat16* ag = a_ptr + (long long)grp * p.G * img_a + a_g * 8;
        const __nv_bfloat16* dg = dy_ptr + (long long)grp * p.G * img_d + d_g * 8;
        const uint32_t st0 = s_u32(ring + stage * stage_bytes);
        if (a_on) {
            const int* t = table + j * sub + a_row0;
            uint32_t dst = st0 + dy_bytes + a_g * 16 + a_row0 * apitch;
            for (int row = a_row0; row < rows_a; row += a_step, t += a_step, dst += a_step * apitch) {
                const int pix = *t;                                // padding: read nothing, write zeros
                cp_async16(dst, ag + (long long)max(pix, 0) * C, pix >= 0 ? 16u : 0u);
            }
        }
        if (d_on) {
            const int* t = stuffed ? dtable + j * sub + d_row0 : table + j * sub + halo + d_row0;
            uint32_t dst = st0 + d_g * 16 + d_row0 * dpitch;
            for (int row = d_row0; row < sub; row += d_step, t += d_step, dst += d_step * dpitch) {
                const int pix = *t;
                cp_async16(dst, dg + (long long)max(pix, 0) * K, pix >= 0 ? 16u : 0u);
            }
        }
    };

    const uint32_t b_lane = (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * apitch + (lane >> 4) * 16;
    // ---- the column pairs of this warp: byte offset of (tap shift, 16 channels) in the activation window.  A warp with
    // fewer than PPW pairs repeats its first one (no branch in the inner loop) and drops those sums at the end.
    const int cpairs = C / 16, NP = ntap * cpairs;
    uint32_t b_off[PPW];
#pragma unroll
    for (int e = 0; e < PPW; ++e) {
        int q = warp_n * PPW + e; if (q >= NP) q = 0;
        const int tt = q / cpairs, cp = q - tt * cpairs, tap = tap0 + tt, r = tap / p.ksz, s = tap - r * p.ksz;
        b_off[e] = (uint32_t)((r * Wp + s) * apitch + cp * 32) + b_lane;
    }
    float acc[PPW][2][MB][4];
#pragma unroll
    for (int e = 0; e < PPW; ++e)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int m = 0; m < MB; ++m) { acc[e][h][m][0] = acc[e][h][m][1] = acc[e][h][m][2] = acc[e][h][m][3] = 0.f; }
    // A = dy^T (stored [position][k], transposed on load); B = activations (stored [position][c], transposed on load)
    const uint32_t a_lane = (uint32_t)((lane & 7) + ((lane >> 4) & 1) * 8) * dpitch + ((lane >> 3) & 1) * 16;
    const int ksteps = sub / 16;

    __syncthreads();                                              // table complete
    pdl_wait();                                                   // from here on: tensors the previous kernel may have written
    const int units = p.units;
    int nxt = split;
    for (int st = 0; st < stages - 1; ++st) { if (nxt < units) issue(nxt, st); cp_async_commit(); nxt += p.splits; }
    int stage = 0;
    for (int unit = split; unit < units; unit += p.splits) {
        { const int ps = stage == 0 ? stages - 1 : stage - 1; if (nxt < units) issue(nxt, ps); cp_async_commit(); nxt += p.splits; }
        if (stages == 2) cp_async_wait<1>(); else if (stages == 3) cp_async_wait<2>(); else cp_async_wait<3>();
        __syncthreads();
        const uint32_t st0 = s_u32(ring + stage * stage_bytes);
        uint32_t dy_row = st0 + a_lane + (uint32_t)(warp_p * 16) * dpitch, b_row = st0 + dy_bytes + (uint32_t)(warp_p * 16) * apitch;
        for (int ks = warp_p; ks < ksteps; ks += WP, dy_row += WP * 16 * dpitch, b_row += WP * 16 * apitch) {
            uint32_t af[MB][4];
#pragma unroll
            for (int m = 0; m < MB; ++m) ldsm_x4_t(dy_row + m * 32, af[m][0], af[m][1], af[m][2], af[m][3]);
#pragma unroll
            for (int e = 0; e < PPW; ++e) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(b_row + b_off[e], b0, b1, b2, b3);
#pragma unroll
                for (int m = 0; m < MB; ++m) {
                    mma16816(acc[e][0][m], af[m][0], af[m][1], af[m][2], af[m][3], b0, b1);
                    mma16816(acc[e][1][m], af[m][0], af[m][1], af[m][2], af[m][3], b2, b3);
                }
            }
        }
        __syncthreads();
        stage = stage + 1 == stages ? 0 : stage + 1;
    }
    cp_async_wait<0>();
    __syncthreads();
    // ---- add the WP partial sums in a fixed order: red[warp_p][tap][k][c]; thread (g8, t4) holds rows g8, g8+8, columns 2*t4, +1
    float* red = reinterpret_cast<float*>(sm);
    const int per = ntap * K * C;
    const int g8 = lane >> 2, t4 = lane & 3;
#pragma unroll
    for (int e = 0; e < PPW; ++e) {
        const int q = warp_n * PPW + e;
        if (q >= NP) continue;
        const int tt = q / cpairs, cp = q - tt * cpairs;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int m = 0; m < MB; ++m)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int k = m * 16 + g8 + half * 8, c = cp * 16 + h * 8 + t4 * 2;
                    *reinterpret_cast<float2*>(red + (long long)warp_p * per + (tt * K + k) * C + c) = make_float2(acc[e][h][m][half * 2], acc[e][h][m][half * 2 + 1]);
                }
    }
    __syncthreads();
    float* dst = p.partial + ((long long)split * p.taps + tap0) * K * C;
    for (int i = tid * 4; i < per; i += MMA_THREADS * 4) {           // per is a multiple of 256; four sums per thread and access
        float4 s = *reinterpret_cast<const float4*>(red + i);
        for (int w = 1; w < WP; ++w) { const float4 v = *reinterpret_cast<const float4*>(red + (long long)w * per + i); s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
        *reinterpret_cast<float4*>(dst + i) = s;
    }
}

// out[k][t][c] = sum over splits of partial[split][t][k][c], in a fixed order: a block owns 32 consecutive elements,
// warp w adds the splits w, w+8, ... (ascending), then the 8 sums are added in warp order.
__global__ void __launch_bounds__(256) wgrad_mma_reduce_kernel(const MmaWgradProb* __restrict__ probs) {
    pdl_trigger();
    pdl_wait();                                                   // launched programmatically behind the kernel that writes the partial sums
    const MmaWgradProb& p = probs[blockIdx.y];
    const int n = p.taps * p.K * p.C, splits = p.splits, taps = p.taps, K = p.K, C = p.C;
    const float* __restrict__ partial = p.partial;
    __shared__ float red[8][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int base = blockIdx.x * 32; base < n; base += gridDim.x * 32) {
        const int i = base + lane;                                // n is a multiple of 256
        float s = 0.f;
#pragma unroll 8
        for (int sp = warp; sp < splits; sp += 8) s += partial[(long long)sp * n + i];
        red[warp][lane] = s;
        __syncthreads();
        if (warp == 0) {
            float t = red[0][lane];
#pragma unroll
            for (int w = 1; w < 8; ++w) t += red[w][lane];
            const int c = i % C, r = i / C, k = r % K, tp = r / K;
            if (c < p.out_cols) p.out[((long long)k * taps + tp) * p.out_ld + c] = t;
        }
        __syncthreads();
    }
}

struct MmaWgGeom { int Hp, Wp, G, n_groups, gpos, sub, subs, units, table_rows, tap_groups, taps_per_group, splits, wn, ppw, stages, variant; size_t smem, partial_bytes; };

static bool mma_wg_geometry(const ConvProb& p, int target_ctas, MmaWgGeom& g) {
    if (p.stride != 1 || (p.ksz != 1 && p.ksz != 3)) return false;
    if (p.C % 16 || p.K % 16 || p.C > 64 || p.K > 64 || p.N < 1) return false;
    if (((uintptr_t)p.act | (uintptr_t)p.wgt) & 15) return false;
    const int taps = p.ksz * p.ksz, pad = p.ksz / 2, MB = p.K / 16, cpairs = p.C / 16;
    g.Hp = p.H + pad; g.Wp = p.W + pad;
    if (g.Hp < 2 || g.Wp < 2) return false;
    const int ppi = g.Hp * g.Wp, halo = pad * g.Wp + pad;
    // taps per CTA and the warp grid: the fewest column splits whose accumulators still fit the registers
    static const int ppw_set[] = {1, 2, 3, 5, 9, 12};
    g.wn = 0;
    for (int tpg : {taps, 3, 1}) {
        if (tpg > taps) continue;
        for (int wn : {1, 2, 4, 8}) {
            const int need = (tpg * cpairs + wn - 1) / wn;
            int ppw = 0; for (int c : ppw_set) if (c >= need) { ppw = c; break; }
            if (ppw && MB * ppw <= 12) { g.wn = wn; g.ppw = ppw; g.taps_per_group = tpg; break; }
        }
        if (g.wn) break;
    }
    if (!g.wn) return false;
    g.tap_groups = (taps + g.taps_per_group - 1) / g.taps_per_group;
    const int quantum = 16 * (8 / g.wn), dpitch = p.K * 2 + 16, apitch = p.C * 2 + 16;
    const size_t red_bytes = (size_t)(8 / g.wn) * g.taps_per_group * p.K * p.C * 4;
    // images per group and positions per piece: little padding of the last piece, pieces not too small
    double best = 1e30; g.sub = 0;
    for (int G = 1; G <= std::min(p.N, 64); ++G) {
        if (p.N % G) continue;
        const int gpos = G * ppi;
        if (gpos + 2 * halo + 512 > 8192) break;
        for (int sub = quantum; sub <= 512; sub += quantum) {
            const int subs = (gpos + sub - 1) / sub;
            const size_t table = (size_t)(((subs * sub + 2 * halo) * 4 + 127) & ~127) + (p.dy_sub == 2 ? (size_t)((subs * sub * 4 + 127) & ~127) : 0);
            const size_t stage = (size_t)((sub * dpitch + 127) & ~127) + (size_t)(((sub + 2 * halo) * apitch + 127) & ~127);
            int stages = 3; if (table + 3 * stage > 150 * 1024) stages = 2;
            if (table + stages * stage + 64 > 200 * 1024) continue;
            const double cost = (double)subs * sub / gpos * (1.0 + 48.0 / sub);
            if (cost < best) { best = cost; g.G = G; g.gpos = gpos; g.sub = sub; g.subs = subs; g.stages = stages; g.smem = std::max(table + stages * stage, red_bytes) + 64; }
        }
    }
    if (!g.sub || g.smem > 200 * 1024) return false;
    g.n_groups = p.N / g.G; g.units = g.n_groups * g.subs; g.table_rows = g.subs * g.sub + 2 * halo;
    const int per_sm = g.smem <= 100 * 1024 ? 2 : 1;
    int want = std::max(1, target_ctas * per_sm / 2 / g.tap_groups); if (want > g.units) want = g.units; if (want > 512) want = 512;
    g.splits = want;
    g.partial_bytes = (size_t)g.splits * taps * p.K * p.C * 4;
    g.variant = MB + 8 * g.ppw;
    return true;
}
bool conv_wgrad_mma_supported(const ConvProb& p, int target_ctas, size_t* partial_bytes) {
    MmaWgGeom g; if (!mma_wg_geometry(p, target_ctas, g)) return false;
    if (partial_bytes) *partial_bytes = g.partial_bytes;
    return true;
}
int conv_wgrad_mma_pick_variant(const ConvProb& p, int target_ctas) { MmaWgGeom g; return mma_wg_geometry(p, target_ctas, g) ? g.variant : 0; }
// p.act = a, p.wgt = dy, p.out = dw (fp32), p.partial = workspace
bool conv_wgrad_mma_fill(const ConvProb& p, int target_ctas, void* host) {
    MmaWgGeom g; if (!mma_wg_geometry(p, target_ctas, g)) return false;
    MmaWgradProb t; memset(&t, 0, sizeof(t));
    t.dy = (const __nv_bfloat16*)p.wgt; t.a = (const __nv_bfloat16*)p.act; t.partial = p.partial; t.out = (float*)p.out;
    t.K = p.K; t.C = p.C; t.H = p.H; t.W = p.W; t.Hp = g.Hp; t.Wp = g.Wp; t.ksz = p.ksz; t.taps = p.ksz * p.ksz;
    t.G = g.G; t.n_groups = g.n_groups; t.gpos = g.gpos; t.sub = g.sub; t.subs = g.subs; t.units = g.units; t.table_rows = g.table_rows;
    t.tap_groups = g.tap_groups; t.taps_per_group = g.taps_per_group; t.splits = g.splits; t.wn = g.wn; t.stages = g.stages; t.variant = g.variant;
    t.inv_wp = (unsigned)((1ull << 32) / (unsigned)g.Wp + 1); t.inv_hp = (unsigned)((1ull << 32) / (unsigned)g.Hp + 1);
    t.smem_bytes = (int)g.smem;
    t.out_ld = p.C; t.out_cols = p.C;
    t.ds = p.dy_sub == 2 ? 2 : 1; t.dP = p.dy_P; t.dQ = p.dy_Q;
    if (p.wg_ld > 0 && p.ksz == 1) { t.out_ld = p.wg_ld; t.out_cols = p.wg_cols; }
    memcpy(host, &t, sizeof(t));
    return true;
}
size_t conv_wgrad_mma_prob_bytes() { return sizeof(MmaWgradProb); }
int conv_wgrad_mma_ctas(const void* h) { const MmaWgradProb* t = (const MmaWgradProb*)h; return t->tap_groups * t->splits; }
size_t conv_wgrad_mma_smem(const void* h) { return (size_t)((const MmaWgradProb*)h)->smem_bytes; }
long long conv_wgrad_mma_out_elems(const void* h) { const MmaWgradProb* t = (const MmaWgradProb*)h; return (long long)t->taps * t->K * t->C; }

template <int MB, int PPW>
static void launch_wg_inst(const void* d, dim3 grid, size_t smem, bool pdl, cudaStream_t s) {
    static bool configured = false;
    if (!configured) { cudaFuncSetAttribute(conv_wgrad_mma_kernel<MB, PPW>, cudaFuncAttributeMaxDynamicSharedMemorySize, 202 * 1024); configured = true; }
    launch_pdl(conv_wgrad_mma_kernel<MB, PPW>, grid, smem, s, pdl, (const MmaWgradProb*)d);
}
// all problems of one launch share the variant (output channels / 16 + 8 * column pairs per warp)
void launch_conv_wgrad_mma_probs(const void* d, int nprob, int max_ctas, size_t max_smem, long long max_out, int variant, cudaStream_t s, bool pdl) {
    const dim3 grid(max_ctas, nprob);
    const int mb = variant & 7, ppw = (variant >> 3) & 31;
#define WG_CASE(M, P) if (mb == M && ppw == P) launch_wg_inst<M, P>(d, grid, max_smem, pdl, s); else
    WG_CASE(1, 1) WG_CASE(1, 2) WG_CASE(1, 3) WG_CASE(1, 5) WG_CASE(1, 9) WG_CASE(1, 12)
    WG_CASE(2, 1) WG_CASE(2, 2) WG_CASE(2, 3) WG_CASE(2, 5)
    WG_CASE(3, 1) WG_CASE(3, 2) WG_CASE(3, 3)
    WG_CASE(4, 1) WG_CASE(4, 2) WG_CASE(4, 3)
    return;
#undef WG_CASE
    long long gx = (max_out + 31) / 32; if (gx > 1184) gx = 1184; if (gx < 1) gx = 1;
    launch_pdl(wgrad_mma_reduce_kernel, dim3((unsigned)gx, nprob), 0, s, true, (const MmaWgradProb*)d);
}

}  // namespace resist
