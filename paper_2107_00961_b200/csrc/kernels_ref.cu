// CUDA-core kernel family: every layer of the sub-ResNet step for storage type T = float or bf16,
// fp32 arithmetic.  It is the whole path of the fp32 mode, and in bf16 mode it runs whatever the
// tensor-core kernels do not take (3-channel stems, odd shapes) and the small head/loss kernels.
// All reductions have a fixed order: results are reproducible run to run.
#include <algorithm>
#include <cooperative_groups.h>
#include "internal.h"

namespace cg = cooperative_groups;
namespace resist {

template <class T> __device__ __forceinline__ float ldf(const void* p, long long i);
template <> __device__ __forceinline__ float ldf<float>(const void* p, long long i) { return ((const float*)p)[i]; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const void* p, long long i) {
    return __bfloat162float(((const __nv_bfloat16*)p)[i]);
}
template <class T> __device__ __forceinline__ void stf(void* p, long long i, float v);
template <> __device__ __forceinline__ void stf<float>(void* p, long long i, float v) { ((float*)p)[i] = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(void* p, long long i, float v) {
    ((__nv_bfloat16*)p)[i] = __float2bfloat16_rn(v);
}

// ------------------------------------------------------------------------------------------------
// Implicit-GEMM convolution on CUDA cores: 64x64 output tile, 16-deep slices, 256 threads, 4x4 per thread.
//   forward: rows = output pixels (n,p,q), cols = output channels, reduction = (r,s,c)
//   dgrad:   rows = input pixels (n,h,w),  cols = input channels,  reduction = (r,s,k)
//   wgrad:   rows = output channels,       cols = (r,s,c),         reduction = output pixels; split over
//            `splits` CTAs along the reduction, partial sums reduced afterwards in a fixed order.
// ------------------------------------------------------------------------------------------------
constexpr int BM = 64, BN = 64, BK = 16;

template <class T, int MODE>
__device__ __forceinline__ float load_a(const ConvProb& p, int row, int kk) {
    if (row >= p.M || kk >= p.Kred) return 0.f;
    if (MODE == CONV_FWD) {
        int q = row % p.Q, t = row / p.Q, pp = t % p.P, n = t / p.P;
        int c = kk % p.C, t2 = kk / p.C, s = t2 % p.ksz, r = t2 / p.ksz;
        int h = pp * p.stride + r - p.pad, x = q * p.stride + s - p.pad;
        if (h < 0 || h >= p.H || x < 0 || x >= p.W) return 0.f;
        return ldf<T>(p.act, (((long long)n * p.H + h) * p.W + x) * p.C + c);
    } else if (MODE == CONV_DGRAD) {
        int x = row % p.W, t = row / p.W, h = t % p.H, n = t / p.H;
        int ko = kk % p.K, t2 = kk / p.K, s = t2 % p.ksz, r = t2 / p.ksz;
        int ph = h + p.pad - r, qx = x + p.pad - s;
        if (ph < 0 || qx < 0 || ph % p.stride || qx % p.stride) return 0.f;
        int pp = ph / p.stride, q = qx / p.stride;
        if (pp >= p.P || q >= p.Q) return 0.f;
        return ldf<T>(p.act, (((long long)n * p.P + pp) * p.Q + q) * p.K + ko);
    } else {   // wgrad: A[ko, t] = dy[t, ko]
        return ldf<T>(p.wgt, (long long)kk * p.K + row);
    }
}
template <class T, int MODE>
__device__ __forceinline__ float load_b(const ConvProb& p, int kk, int col) {
    if (col >= p.Ncol || kk >= p.Kred) return 0.f;
    if (MODE == CONV_FWD) {
        return ldf<T>(p.wgt, (long long)col * p.Kred + kk);
    } else if (MODE == CONV_DGRAD) {
        int ko = kk % p.K, t2 = kk / p.K, s = t2 % p.ksz, r = t2 / p.ksz;
        return ldf<T>(p.wgt, (((long long)ko * p.ksz + r) * p.ksz + s) * p.C + col);
    } else {   // wgrad: B[t, (r,s,c)] = a[n, p*stride+r-pad, q*stride+s-pad, c]
        int q = kk % p.Q, t = kk / p.Q, pp = t % p.P, n = t / p.P;
        int c = col % p.C, t2 = col / p.C, s = t2 % p.ksz, r = t2 / p.ksz;
        int h = pp * p.stride + r - p.pad, x = q * p.stride + s - p.pad;
        if (h < 0 || h >= p.H || x < 0 || x >= p.W) return 0.f;
        return ldf<T>(p.act, (((long long)n * p.H + h) * p.W + x) * p.C + c);
    }
}

template <class T, int MODE>
__global__ void __launch_bounds__(256) conv_ref_kernel(const ConvProb* __restrict__ probs) {
    const ConvProb& p = probs[blockIdx.y];
    const int tiles = p.tiles_m * p.tiles_n;
    int tile = blockIdx.x;
    if (tile >= tiles * p.splits) return;
    const int split = tile / tiles; tile -= split * tiles;
    const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
    float acc[4][4] = {};
    const int kt0 = split * p.ktiles_per_split;
    int kt1 = kt0 + p.ktiles_per_split;
    const int ktiles = (p.Kred + BK - 1) / BK;
    if (kt1 > ktiles) kt1 = ktiles;
    for (int kt = kt0; kt < kt1; ++kt) {
        const int k0 = kt * BK;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int e = tid + 256 * i;
            if (MODE == CONV_WGRAD) { int r = e % BM, kc = e / BM; As[kc][r] = load_a<T, MODE>(p, tm * BM + r, k0 + kc); }
            else { int kc = e % BK, r = e / BK; As[kc][r] = load_a<T, MODE>(p, tm * BM + r, k0 + kc); }
            if (MODE == CONV_FWD) { int kc = e % BK, c = e / BK; Bs[kc][c] = load_b<T, MODE>(p, k0 + kc, tn * BN + c); }
            else { int c = e % BN, kc = e / BN; Bs[kc][c] = load_b<T, MODE>(p, k0 + kc, tn * BN + c); }
        }
        __syncthreads();
#pragma unroll
        for (int kc = 0; kc < BK; ++kc) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[kc][ty * 4 + i]; b[i] = Bs[kc][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = tm * BM + ty * 4 + i;
        if (row >= p.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = tn * BN + tx * 4 + j;
            if (col >= p.Ncol) continue;
            const long long o = (long long)row * p.Ncol + col;
            if (MODE == CONV_WGRAD) {
                if (p.splits > 1) p.partial[(long long)split * p.M * p.Ncol + o] = acc[i][j];
                else ((float*)p.out)[o] = acc[i][j];
            } else {
                float v = acc[i][j] * p.scale;
                if (p.add) v += ldf<T>(p.add, o);
                stf<T>(p.out, o, v);
            }
        }
    }
}

__global__ void splitk_reduce_kernel(const ConvProb* __restrict__ probs) {
    const ConvProb& p = probs[blockIdx.y];
    if (p.splits <= 1) return;
    const long long n = (long long)p.M * p.Ncol;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        float s = 0.f;
        for (int k = 0; k < p.splits; ++k) s += p.partial[(long long)k * n + i];
        ((float*)p.out)[i] = s;
    }
}

void launch_conv_ref(const ConvProb* d, int nprob, int max_tiles, int mode, bool bf16, cudaStream_t s) {
    dim3 g(max_tiles, nprob);
    if (!bf16) {
        if (mode == CONV_FWD) conv_ref_kernel<float, CONV_FWD><<<g, 256, 0, s>>>(d);
        else if (mode == CONV_DGRAD) conv_ref_kernel<float, CONV_DGRAD><<<g, 256, 0, s>>>(d);
        else conv_ref_kernel<float, CONV_WGRAD><<<g, 256, 0, s>>>(d);
    } else {
        if (mode == CONV_FWD) conv_ref_kernel<__nv_bfloat16, CONV_FWD><<<g, 256, 0, s>>>(d);
        else if (mode == CONV_DGRAD) conv_ref_kernel<__nv_bfloat16, CONV_DGRAD><<<g, 256, 0, s>>>(d);
        else conv_ref_kernel<__nv_bfloat16, CONV_WGRAD><<<g, 256, 0, s>>>(d);
    }
}
void launch_splitk_reduce(const ConvProb* d, int nprob, int max_elems, cudaStream_t s) {
    int gx = (max_elems + 255) / 256; if (gx > 1184) gx = 1184; if (gx < 1) gx = 1;
    splitk_reduce_kernel<<<dim3(gx, nprob), 256, 0, s>>>(d);
}

// ------------------------------------------------------------------------------------------------
// Batch normalisation + ReLU.  Statistics: each CTA reduces `rows_per_chunk` rows of all C channels
// (fp32 per thread, fp64 across threads), a finalise kernel adds the chunk partials in order.
// ------------------------------------------------------------------------------------------------

// ---- bf16 fast path: 16-byte accesses, a thread owns 8 consecutive channels (one group) and every (256/G)-th row
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) { f[2 * k] = __uint_as_float(w[k] << 16); f[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u); }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) { __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]); w[k] = *reinterpret_cast<uint32_t*>(&h); }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

template <int MODE>
__device__ void bn_reduce_vec(const BnProb& p) {
    __shared__ float sm[256][17];
    const int C = p.C, G = C >> 3, R = 256 / G;
    const int g = threadIdx.x % G, r = threadIdx.x / G;
    const long long r0 = (long long)blockIdx.x * p.rows_per_chunk;
    long long r1 = r0 + p.rows_per_chunk; if (r1 > p.m) r1 = p.m;
    float s0[8], s1[8], sh[8], mean[8], istd[8], ga[8], be[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { s0[j] = 0.f; s1[j] = 0.f; }
    if (MODE == 0) { unpack8(*reinterpret_cast<const uint4*>((const __nv_bfloat16*)p.x + g * 8), sh); }
    else {
#pragma unroll
        for (int j = 0; j < 8; ++j) { const int c = g * 8 + j; mean[j] = p.stat[c]; istd[j] = p.stat[C + c]; ga[j] = p.gamma[c]; be[j] = p.beta[c]; }
    }
    const uint4* xv = reinterpret_cast<const uint4*>(p.x);
    const uint4* dv = reinterpret_cast<const uint4*>(p.da);
    // U rows of loads in flight per thread (backward: x and dy, so six rows = twelve 16-byte loads; forward: eight rows); the rows
    // are still added in ascending order
    constexpr int U = MODE == 1 ? 6 : 8;
    for (long long row = r0 + r; row < r1; row += U * R) {
        uint4 xs[U], ds[MODE == 1 ? U : 1];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long rr = row + (long long)u * R;
            if (rr < r1) { xs[u] = __ldg(xv + rr * G + g); if (MODE == 1) ds[u] = __ldg(dv + rr * G + g); }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (row + (long long)u * R >= r1) break;
            float x[8]; unpack8(xs[u], x);
            if (MODE == 0) {
#pragma unroll
                for (int j = 0; j < 8; ++j) { const float d = x[j] - sh[j]; s0[j] += d; s1[j] += d * d; }
            } else {
                float d[8]; unpack8(ds[u], d);
#pragma unroll
                for (int j = 0; j < 8; ++j) { const float xh = (x[j] - mean[j]) * istd[j]; const float dz = (xh * ga[j] + be[j] > 0.f) ? d[j] : 0.f; s0[j] += dz; s1[j] += dz * xh; }
            }
        }
    }
    // lanes of a warp that own the same channel group: fixed-order butterfly in fp32
    if (G < 32) {
        for (int off = 16; off >= G; off >>= 1) {
#pragma unroll
            for (int j = 0; j < 8; ++j) { s0[j] += __shfl_down_sync(0xffffffffu, s0[j], off); s1[j] += __shfl_down_sync(0xffffffffu, s1[j], off); }
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) { sm[threadIdx.x][j] = s0[j]; sm[threadIdx.x][8 + j] = s1[j]; }
    __syncthreads();
    if ((int)threadIdx.x < C) {
        const int c = threadIdx.x, cg = c >> 3, j = c & 7;
        double a0 = 0.0, a1 = 0.0;
        if (G < 32) { for (int w = 0; w < 8; ++w) { a0 += sm[w * 32 + cg][j]; a1 += sm[w * 32 + cg][8 + j]; } }
        else { for (int k = 0; k < R; ++k) { a0 += sm[cg + G * k][j]; a1 += sm[cg + G * k][8 + j]; } }
        p.partial[((long long)blockIdx.x * 2 + 0) * C + c] = a0;
        p.partial[((long long)blockIdx.x * 2 + 1) * C + c] = a1;
    }
    // more than 256 channels: the remaining ones, 256 at a time
    for (int c = threadIdx.x + 256; c < C; c += 256) {
        const int cg = c >> 3, j = c & 7;
        double a0 = 0.0, a1 = 0.0;
        for (int k = 0; k < R; ++k) { a0 += sm[cg + G * k][j]; a1 += sm[cg + G * k][8 + j]; }
        p.partial[((long long)blockIdx.x * 2 + 0) * C + c] = a0;
        p.partial[((long long)blockIdx.x * 2 + 1) * C + c] = a1;
    }
}

// Streaming form of the elementwise pass (bf16 vector path; stat: [4][C] as BnProb::stat, in global or shared memory): a thread keeps ONE group of 8 channels for all its rows, so the
// per-channel constants are loaded once into registers and the loop is loads, arithmetic and a store; a CTA takes at least 16 passes
// of 256 / G rows (32768 elements), four rows of loads in flight per thread.  MODE 0: a = relu(bn(x)); MODE 1: dx (+ add).
template <int MODE>
__device__ void bn_stream_vec(const BnProb& p, const float* __restrict__ stat) {
    const int C = p.C, G = C >> 3, R = 256 / G;
    const int g = threadIdx.x % G, r = threadIdx.x / G;
    // the grid's CTAs share the rows evenly, in whole passes of 4 * R rows (at least 16 passes of R rows each)
    long long rows_per_cta = (p.m + gridDim.x - 1) / gridDim.x;
    rows_per_cta = (rows_per_cta + 4 * R - 1) / (4 * R) * (4 * R); if (rows_per_cta < 16 * R) rows_per_cta = 16 * R;
    const long long r0 = (long long)blockIdx.x * rows_per_cta;
    if (r0 >= p.m) return;
    const long long r1 = r0 + rows_per_cta < p.m ? r0 + rows_per_cta : p.m;
    float mean[8], istd[8], ga[8], be[8], sb[8], sg[8];
    const float inv_m = 1.f / (float)p.m;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int c = g * 8 + j;
        mean[j] = stat[c]; istd[j] = stat[C + c]; ga[j] = p.gamma[c]; be[j] = p.beta[c];
        if (MODE == 1) { sb[j] = stat[2 * C + c] * inv_m; sg[j] = stat[3 * C + c] * inv_m; }
    }
    const uint4* xv = reinterpret_cast<const uint4*>(p.x);
    const uint4* dv = reinterpret_cast<const uint4*>(p.da);
    const uint4* av = reinterpret_cast<const uint4*>(p.add);
    uint4* ov = reinterpret_cast<uint4*>(MODE == 0 ? p.a : p.dx);
    for (long long row = r0 + r; row < r1; row += 4 * R) {
        uint4 xs[4], ds[4], as[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long rr = row + (long long)u * R;
            if (rr < r1) {
                xs[u] = __ldg(xv + rr * G + g);
                if (MODE == 1) { ds[u] = __ldg(dv + rr * G + g); if (av) as[u] = __ldg(av + rr * G + g); }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long rr = row + (long long)u * R;
            if (rr < r1) {
                float x[8], o[8]; unpack8(xs[u], x);
                if (MODE == 0) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) { const float z = (x[j] - mean[j]) * istd[j] * ga[j] + be[j]; o[j] = z > 0.f ? z : 0.f; }
                } else {
                    float d[8]; unpack8(ds[u], d);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float xh = (x[j] - mean[j]) * istd[j];
                        const float dz = (xh * ga[j] + be[j] > 0.f) ? d[j] : 0.f;
                        o[j] = ga[j] * istd[j] * (dz - sb[j] - xh * sg[j]);
                    }
                    if (av) { float ad[8]; unpack8(as[u], ad);
#pragma unroll
                        for (int j = 0; j < 8; ++j) o[j] += ad[j]; }
                }
                ov[rr * G + g] = pack8(o);
            }
        }
    }
}

// MODE 0: sums of x and x^2.  MODE 1: sums of dz and dz*xhat (backward).
template <class T, int MODE>
__global__ void __launch_bounds__(256) bn_reduce_kernel(const BnProb* __restrict__ probs) {
    const BnProb& p = probs[blockIdx.y];
    if ((int)blockIdx.x >= p.chunks || p.eval) return;
    if (p.vec) { bn_reduce_vec<MODE>(p); return; }
    __shared__ double part[2][256];
    const int C = p.C, nl = C < 256 ? C : 256, R = 256 / nl;
    const int rg = threadIdx.x / nl, lane = threadIdx.x % nl;
    const long long r0 = (long long)blockIdx.x * p.rows_per_chunk;
    long long r1 = r0 + p.rows_per_chunk; if (r1 > p.m) r1 = p.m;
    for (int cb = 0; cb < C; cb += nl) {
        const int c = cb + lane;
        float s0 = 0.f, s1 = 0.f;
        if (rg < R && c < C) {
            float mean = 0.f, istd = 0.f, g = 0.f, b = 0.f, shift = 0.f;
            if (MODE == 1) { mean = p.stat[c]; istd = p.stat[C + c]; g = p.gamma[c]; b = p.beta[c]; }
            else shift = ldf<T>(p.x, c);      // sums of (x - x[0,c]): no cancellation when |mean| >> std
            for (long long r = r0 + rg; r < r1; r += R) {
                float x = ldf<T>(p.x, r * C + c);
                if (MODE == 0) { x -= shift; s0 += x; s1 += x * x; }
                else {
                    float xh = (x - mean) * istd;
                    float dz = (xh * g + b > 0.f) ? ldf<T>(p.da, r * C + c) : 0.f;
                    s0 += dz; s1 += dz * xh;
                }
            }
        }
        __syncthreads();
        part[0][threadIdx.x] = s0; part[1][threadIdx.x] = s1;
        __syncthreads();
        if (rg == 0 && c < C) {
            double a0 = 0.0, a1 = 0.0;
            for (int k = 0; k < R; ++k) { a0 += part[0][k * nl + lane]; a1 += part[1][k * nl + lane]; }
            p.partial[((long long)blockIdx.x * 2 + 0) * C + c] = a0;
            p.partial[((long long)blockIdx.x * 2 + 1) * C + c] = a1;
        }
    }
}

template <class T, int MODE>
__global__ void bn_finalize_kernel(const BnProb* __restrict__ probs) {
    // one warp per channel: lane l adds chunks l, l+32, ... in order, then a fixed butterfly over the lanes
    const BnProb& p = probs[blockIdx.y];
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (c >= p.C) return;
    if (p.eval) {
        if (MODE == 0 && lane == 0) { p.stat[c] = p.run_mean[c]; p.stat[p.C + c] = (float)(1.0 / sqrt((double)p.run_var[c] + (double)p.eps)); }
        return;
    }
    double a0 = 0.0, a1 = 0.0;
    for (int k = lane; k < p.chunks; k += 32) { a0 += p.partial[((long long)k * 2 + 0) * p.C + c]; a1 += p.partial[((long long)k * 2 + 1) * p.C + c]; }
    for (int d = 16; d; d >>= 1) { a0 += __shfl_xor_sync(0xffffffffu, a0, d); a1 += __shfl_xor_sync(0xffffffffu, a1, d); }
    if (lane != 0) return;
    if (MODE == 0) {
        const double m = (double)p.m, dm = a0 / m;                 // sums are of x - x[0,c]
        double var = a1 / m - dm * dm; if (var < 0.0) var = 0.0;
        const double mean = dm + (double)ldf<T>(p.x, c);
        p.stat[c] = (float)mean;
        p.stat[p.C + c] = (float)(1.0 / sqrt(var + (double)p.eps));
        if (p.run_mean) {
            const double unb = p.m > 1 ? var * m / (m - 1.0) : var, mo = (double)p.momentum;
            p.run_mean[c] = (float)((1.0 - mo) * (double)p.run_mean[c] + mo * mean);
            p.run_var[c] = (float)((1.0 - mo) * (double)p.run_var[c] + mo * unb);
        }
    } else {
        p.stat[2 * p.C + c] = (float)a0; p.stat[3 * p.C + c] = (float)a1;
        p.dbeta[c] = (float)a0; p.dgamma[c] = (float)a1;
    }
}

template <class T>
__global__ void __launch_bounds__(256) bn_apply_kernel(const BnProb* __restrict__ probs) {
    const BnProb& p = probs[blockIdx.y];
    if (p.vec) { bn_stream_vec<0>(p, p.stat); return; }
    const long long n = p.m * p.C;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % p.C);
        float z = (ldf<T>(p.x, i) - p.stat[c]) * p.stat[p.C + c] * p.gamma[c] + p.beta[c];
        stf<T>(p.a, i, z > 0.f ? z : 0.f);
    }
}

template <class T>
__global__ void __launch_bounds__(256, 2) bn_bwd_apply_kernel(const BnProb* __restrict__ probs) {
    const BnProb& p = probs[blockIdx.y];
    if (p.vec) { bn_stream_vec<1>(p, p.stat); return; }
    const long long n = p.m * p.C;
    const float inv_m = 1.f / (float)p.m;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % p.C);
        const float istd = p.stat[p.C + c], g = p.gamma[c];
        const float xh = (ldf<T>(p.x, i) - p.stat[c]) * istd;
        const float dz = (xh * g + p.beta[c] > 0.f) ? ldf<T>(p.da, i) : 0.f;
        float v = g * istd * (dz - p.stat[2 * p.C + c] * inv_m - xh * p.stat[3 * p.C + c] * inv_m);
        if (p.add) v += ldf<T>(p.add, i);
        stf<T>(p.dx, i, v);
    }
}


// ------------------------------------------------------------------------------------------------ fused BN+ReLU (cooperative)
// One launch per BN layer and direction: partial sums per chunk, a grid-wide barrier, then EVERY CTA adds the
// partials of its problem in the same fixed order (so all CTAs hold identical statistics without a second barrier;
// CTA 0 of the problem also stores them) and takes its share of the elementwise pass, whose re-read of x comes
// from L2.  bf16 vector path, training mode only.
template <int MODE>
__global__ void __launch_bounds__(256, 2) bn_fused_kernel(const BnProb* __restrict__ probs) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a convolution launched behind this kernel may start its prologue
    const BnProb& p = probs[blockIdx.y];
    __shared__ __align__(16) float s_stat[4 * 512];               // callers keep C <= 512
    if ((int)blockIdx.x < p.chunks) bn_reduce_vec<MODE>(p);
    __threadfence();
    cg::this_grid().sync();
    // every CTA adds the partial sums of all chunks in the same fixed order: thread (c, q) adds chunks q, q+Q, ...
    // (independent loads), then thread c adds the Q sums in order
    const int C = p.C;
    __shared__ double s_red[2][256];
    for (int cb = 0; cb < C; cb += 256) {
        const int nl = C - cb < 256 ? C - cb : 256, Q = 256 / nl;
        const int c = cb + (int)threadIdx.x % nl, q = (int)threadIdx.x / nl;
        double a0 = 0.0, a1 = 0.0;
        if (q < Q) {
#pragma unroll 4
            for (int k = q; k < p.chunks; k += Q) { a0 += __ldcg(p.partial + ((long long)k * 2 + 0) * C + c); a1 += __ldcg(p.partial + ((long long)k * 2 + 1) * C + c); }
        }
        __syncthreads();
        s_red[0][threadIdx.x] = a0; s_red[1][threadIdx.x] = a1;
        __syncthreads();
        if (q != 0) continue;
        a0 = 0.0; a1 = 0.0;
        for (int k = 0; k < Q; ++k) { a0 += s_red[0][k * nl + (c - cb)]; a1 += s_red[1][k * nl + (c - cb)]; }
        if (MODE == 0) {
            const double m = (double)p.m, dm = a0 / m;             // sums are of x - x[0,c]
            double var = a1 / m - dm * dm; if (var < 0.0) var = 0.0;
            const double mean = dm + (double)__bfloat162float(((const __nv_bfloat16*)p.x)[c]);
            const float fm = (float)mean, fi = (float)(1.0 / sqrt(var + (double)p.eps));
            s_stat[c] = fm; s_stat[C + c] = fi;
            if (blockIdx.x == 0) {
                p.stat[c] = fm; p.stat[C + c] = fi;
                if (p.run_mean) {
                    const double unb = p.m > 1 ? var * m / (m - 1.0) : var, mo = (double)p.momentum;
                    p.run_mean[c] = (float)((1.0 - mo) * (double)p.run_mean[c] + mo * mean);
                    p.run_var[c] = (float)((1.0 - mo) * (double)p.run_var[c] + mo * unb);
                }
            }
        } else {
            s_stat[c] = p.stat[c]; s_stat[C + c] = p.stat[C + c];
            s_stat[2 * C + c] = (float)a0; s_stat[3 * C + c] = (float)a1;
            if (blockIdx.x == 0) { p.stat[2 * C + c] = (float)a0; p.stat[3 * C + c] = (float)a1; p.dbeta[c] = (float)a0; p.dgamma[c] = (float)a1; }
        }
    }
    __syncthreads();
    bn_stream_vec<MODE>(p, s_stat);
}

// CTAs of the cooperative kernel that can be resident together on this device (its largest grid)
int bn_fused_capacity(int backward) {
    static int cap[2] = {0, 0};
    if (!cap[backward]) {
        int dev = 0, sms = 0, per = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (backward) cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, bn_fused_kernel<1>, 256, 0);
        else cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, bn_fused_kernel<0>, 256, 0);
        cap[backward] = per * sms > 0 ? per * sms : -1;
    }
    return cap[backward];
}
bool launch_bn_fused(const BnProb* d, int nprob, int max_chunks, int backward, cudaStream_t s) {
    if ((long long)max_chunks * nprob > bn_fused_capacity(backward)) return false;
    void* args[] = {(void*)&d};
    const dim3 grid(max_chunks, nprob), block(256);
    const cudaError_t e = backward ? cudaLaunchCooperativeKernel((void*)bn_fused_kernel<1>, grid, block, args, 0, s)
                                   : cudaLaunchCooperativeKernel((void*)bn_fused_kernel<0>, grid, block, args, 0, s);
    return e == cudaSuccess;
}

static int ew_grid(long long n) { long long g = (n + 255) / 256; if (g > 148 * 16) g = 148 * 16; if (g < 1) g = 1; return (int)g; }

void launch_bn_stats(const BnProb* d, int nprob, int max_chunks, int max_c, bool bf16, cudaStream_t s) {
    if (bf16) bn_reduce_kernel<__nv_bfloat16, 0><<<dim3(max_chunks, nprob), 256, 0, s>>>(d);
    else bn_reduce_kernel<float, 0><<<dim3(max_chunks, nprob), 256, 0, s>>>(d);
    if (bf16) bn_finalize_kernel<__nv_bfloat16, 0><<<dim3((max_c + 7) / 8, nprob), 256, 0, s>>>(d);
    else bn_finalize_kernel<float, 0><<<dim3((max_c + 7) / 8, nprob), 256, 0, s>>>(d);
}
// the vector path takes at least 32768 elements per CTA (see bn_stream_vec), and about 16 CTAs per SM over the launch
static int stream_grid(long long n, int nprob) { long long g = (n + 32767) / 32768; const long long cap = std::max(1, 148 * 16 / std::max(1, nprob)); if (g > cap) g = cap; if (g < 1) g = 1; return (int)g; }
void launch_bn_apply(const BnProb* d, int nprob, long long max_elems, bool bf16, cudaStream_t s) {
    if (bf16) bn_apply_kernel<__nv_bfloat16><<<dim3(stream_grid(max_elems, nprob), nprob), 256, 0, s>>>(d);
    else bn_apply_kernel<float><<<dim3(ew_grid(max_elems), nprob), 256, 0, s>>>(d);
}
void launch_bn_bwd_reduce(const BnProb* d, int nprob, int max_chunks, int max_c, bool bf16, cudaStream_t s) {
    if (bf16) bn_reduce_kernel<__nv_bfloat16, 1><<<dim3(max_chunks, nprob), 256, 0, s>>>(d);
    else bn_reduce_kernel<float, 1><<<dim3(max_chunks, nprob), 256, 0, s>>>(d);
    bn_finalize_kernel<float, 1><<<dim3((max_c + 7) / 8, nprob), 256, 0, s>>>(d);
}
void launch_bn_bwd_apply(const BnProb* d, int nprob, long long max_elems, bool bf16, cudaStream_t s) {
    if (bf16) bn_bwd_apply_kernel<__nv_bfloat16><<<dim3(stream_grid(max_elems, nprob), nprob), 256, 0, s>>>(d);
    else bn_bwd_apply_kernel<float><<<dim3(ew_grid(max_elems), nprob), 256, 0, s>>>(d);
}

// ------------------------------------------------------------------------------------------------
// 3x3 stride-2 max-pool (padding 1, padded cells never win; first maximum in row-major window order)
// ------------------------------------------------------------------------------------------------
template <class T>
__global__ void maxpool_fwd_kernel(const PoolProb* __restrict__ probs) {
    const PoolProb& p = probs[blockIdx.y];
    const long long n = (long long)p.N * p.P * p.Q * p.C;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        int c = (int)(i % p.C); long long t = i / p.C; int q = (int)(t % p.Q); t /= p.Q; int pp = (int)(t % p.P); int nn = (int)(t / p.P);
        bool have = false; float best = 0.f; int bi = -1;
        for (int r = 0; r < 3; ++r) { int h = 2 * pp + r - 1; if (h < 0 || h >= p.H) continue;
            for (int s = 0; s < 3; ++s) { int w = 2 * q + s - 1; if (w < 0 || w >= p.W) continue;
                float v = ldf<T>(p.x, (((long long)nn * p.H + h) * p.W + w) * p.C + c);
                if (!have || v > best) { have = true; best = v; bi = h * p.W + w; } } }
        stf<T>(p.y, i, best);
        if (p.arg) p.arg[i] = bi;
    }
}
template <class T>
__global__ void maxpool_bwd_kernel(const PoolProb* __restrict__ probs) {
    const PoolProb& p = probs[blockIdx.y];
    const long long n = (long long)p.N * p.H * p.W * p.C;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        int c = (int)(i % p.C); long long t = i / p.C; int w = (int)(t % p.W); t /= p.W; int h = (int)(t % p.H); int nn = (int)(t / p.H);
        float acc = 0.f;
        for (int pp = h / 2; pp <= (h + 1) / 2; ++pp) { if (pp >= p.P) continue;          // windows with 2p-1 <= h <= 2p+1
            for (int q = w / 2; q <= (w + 1) / 2; ++q) { if (q >= p.Q) continue;
                long long o = (((long long)nn * p.P + pp) * p.Q + q) * p.C + c;
                if (p.arg[o] == h * p.W + w) acc += ldf<T>(p.dy, o); } }
        stf<T>(p.dx, i, acc);
    }
}
void launch_maxpool_fwd(const PoolProb* d, int nprob, long long max_elems, bool bf16, cudaStream_t s) {
    if (bf16) maxpool_fwd_kernel<__nv_bfloat16><<<dim3(ew_grid(max_elems), nprob), 256, 0, s>>>(d);
    else maxpool_fwd_kernel<float><<<dim3(ew_grid(max_elems), nprob), 256, 0, s>>>(d);
}
void launch_maxpool_bwd(const PoolProb* d, int nprob, long long max_elems, bool bf16, cudaStream_t s) {
    if (bf16) maxpool_bwd_kernel<__nv_bfloat16><<<dim3(ew_grid(max_elems), nprob), 256, 0, s>>>(d);
    else maxpool_bwd_kernel<float><<<dim3(ew_grid(max_elems), nprob), 256, 0, s>>>(d);
}

// ------------------------------------------------------------------------------------------------
// Global average pool, linear head, mean softmax cross-entropy and their gradients (fp32 math)
// ------------------------------------------------------------------------------------------------
template <class T>
__global__ void avgpool_kernel(const HeadProb* __restrict__ probs) {
    const HeadProb& p = probs[blockIdx.y];
    const int n = p.B * p.C;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const int c = i % p.C, b = i / p.C;
        float s = 0.f;
        int k = 0;
        for (; k + 8 <= p.HW; k += 8) {                          // eight loads in flight, added in order
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = ldf<T>(p.a, ((long long)b * p.HW + k + u) * p.C + c);
#pragma unroll
            for (int u = 0; u < 8; ++u) s += v[u];
        }
        for (; k < p.HW; ++k) s += ldf<T>(p.a, ((long long)b * p.HW + k) * p.C + c);
        p.pooled[i] = s / (float)p.HW;
    }
}
// one warp per logit
__global__ void head_logits_kernel(const HeadProb* __restrict__ probs) {
    const HeadProb& p = probs[blockIdx.y];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) / 32, lane = threadIdx.x % 32;
    const int nw = gridDim.x * blockDim.x / 32;
    for (int o = warp; o < p.B * p.classes; o += nw) {
        const int k = o % p.classes, b = o / p.classes;
        float s = 0.f;
        for (int c = lane; c < p.C; c += 32) s = fmaf(p.w[(long long)k * p.C + c], p.pooled[(long long)b * p.C + c], s);
        for (int d = 16; d; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
        if (lane == 0) { s += p.b[k]; p.logits[o] = s; if (p.logits_user) p.logits_user[o] = s; }
    }
}
// one CTA per problem; one warp per sample, samples strided over the warps; fixed-order loss sum
__global__ void __launch_bounds__(1024) loss_kernel(const HeadProb* __restrict__ probs) {
    const HeadProb& p = probs[blockIdx.x];
    __shared__ float sl[1024]; __shared__ int sc[1024];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    for (int b = warp; b < p.B; b += (int)(blockDim.x >> 5)) {
        const float* lg = p.logits + (long long)b * p.classes;
        float mx = -INFINITY; int arg = 0x7fffffff;
        for (int k = lane; k < p.classes; k += 32) { float v = lg[k]; if (v > mx) { mx = v; arg = k; } }
        for (int d = 16; d; d >>= 1) {
            float om = __shfl_xor_sync(0xffffffffu, mx, d); int oa = __shfl_xor_sync(0xffffffffu, arg, d);
            if (om > mx || (om == mx && oa < arg)) { mx = om; arg = oa; }
        }
        float se = 0.f;
        for (int k = lane; k < p.classes; k += 32) se += expf(lg[k] - mx);
        for (int d = 16; d; d >>= 1) se += __shfl_xor_sync(0xffffffffu, se, d);
        const float lse = mx + logf(se);
        const int y = p.labels ? p.labels[b] : -1;
        if (p.dlogits)
            for (int k = lane; k < p.classes; k += 32)
                p.dlogits[(long long)b * p.classes + k] = (expf(lg[k] - lse) - (k == y ? 1.f : 0.f)) / (float)p.B;
        if (lane == 0) { sl[b] = y >= 0 ? lse - lg[y] : 0.f; sc[b] = (arg == y); }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f; int c = 0;
        for (int b = 0; b < p.B; ++b) { s += sl[b]; c += sc[b]; }
        s /= (float)p.B;
        if (p.loss) *p.loss = s;
        if (p.loss_user) *p.loss_user = s;
        if (p.correct) *p.correct = c;
    }
}
// one thread per element of dw (neighbouring threads = neighbouring input channels: the loads of `pooled` are coalesced and the
// dlogits value is the same for a whole warp); samples added in order.  The last `classes` threads make the bias gradient.
__global__ void head_bwd_w_kernel(const HeadProb* __restrict__ probs) {
    const HeadProb& p = probs[blockIdx.y];
    const int n = p.classes * p.C;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n + p.classes; i += gridDim.x * blockDim.x) {
        float s = 0.f;
        if (i < n) { const int c = i % p.C, k = i / p.C;
#pragma unroll 4
            for (int b = 0; b < p.B; ++b) s = fmaf(p.dlogits[(long long)b * p.classes + k], p.pooled[(long long)b * p.C + c], s);
            p.dw[i] = s;
        } else { const int k = i - n;
            for (int b = 0; b < p.B; ++b) s += p.dlogits[(long long)b * p.classes + k];
            p.db[k] = s; }
    }
}
__global__ void head_bwd_x_kernel(const HeadProb* __restrict__ probs) {
    const HeadProb& p = probs[blockIdx.y];
    const int n = p.B * p.C;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const int c = i % p.C, b = i / p.C;
        float s = 0.f;
        for (int k = 0; k < p.classes; ++k) s = fmaf(p.dlogits[(long long)b * p.classes + k], p.w[(long long)k * p.C + c], s);
        p.dpooled[i] = s / (float)p.HW;
    }
}
template <class T>
__global__ void avgpool_bwd_kernel(const HeadProb* __restrict__ probs) {
    const HeadProb& p = probs[blockIdx.y];
    const long long n = (long long)p.B * p.HW * p.C;
    if (sizeof(T) == 2 && p.C % 8 == 0 && (((uintptr_t)p.da | (uintptr_t)p.dpooled) & 15) == 0) {   // 8 channels per thread
        const int G = p.C / 8; const long long nv = n / 8;
        for (long long v = blockIdx.x * (long long)blockDim.x + threadIdx.x; v < nv; v += (long long)gridDim.x * blockDim.x) {
            const int g = (int)(v % G); const long long b = v / ((long long)p.HW * G);
            const float4 f0 = *reinterpret_cast<const float4*>(p.dpooled + b * p.C + g * 8), f1 = *reinterpret_cast<const float4*>(p.dpooled + b * p.C + g * 8 + 4);
            const float f[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
            reinterpret_cast<uint4*>(p.da)[v] = pack8(f);
        }
        return;
    }
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % p.C); const long long b = i / ((long long)p.HW * p.C);
        stf<T>(p.da, i, p.dpooled[b * p.C + c]);
    }
}

void launch_head_fwd(const HeadProb* d, int nprob, int maxB, int maxC, int max_classes, bool bf16, cudaStream_t s) {
    if (bf16) avgpool_kernel<__nv_bfloat16><<<dim3(ew_grid((long long)maxB * maxC), nprob), 256, 0, s>>>(d);
    else avgpool_kernel<float><<<dim3(ew_grid((long long)maxB * maxC), nprob), 256, 0, s>>>(d);
    head_logits_kernel<<<dim3(ew_grid((long long)maxB * max_classes * 32), nprob), 256, 0, s>>>(d);
    loss_kernel<<<nprob, 1024, 0, s>>>(d);
}
void launch_head_bwd(const HeadProb* d, int nprob, int maxB, int maxC, int max_classes, long long max_elems,
                     bool bf16, cudaStream_t s) {
    head_bwd_w_kernel<<<dim3(ew_grid((long long)max_classes * (maxC + 1)), nprob), 256, 0, s>>>(d);
    head_bwd_x_kernel<<<dim3(ew_grid((long long)maxB * maxC), nprob), 256, 0, s>>>(d);
    if (bf16) avgpool_bwd_kernel<__nv_bfloat16><<<dim3(ew_grid(max_elems), nprob), 256, 0, s>>>(d);
    else avgpool_bwd_kernel<float><<<dim3(ew_grid(max_elems), nprob), 256, 0, s>>>(d);
}


// ------------------------------------------------------------------------------------------------ im2col (few-channel stem)
// One thread per (output position, 8-column group).  The first K*4 threads also pack the weights.
__global__ void __launch_bounds__(256) im2col_kernel(const ColProb* __restrict__ probs) {
    const ColProb& p = probs[blockIdx.y];
    const __nv_bfloat16* __restrict__ src = (const __nv_bfloat16*)p.src;
    const int cols = p.cols, G = cols >> 3;                       // row pitch in columns (a multiple of 8, at most 256), 8-column groups
    const long long rows = (long long)p.N * p.P * p.Q, total = rows * G;
    // column j of a row = tap (r, s), channel c: the three are looked up, not divided out, for every element
    __shared__ int s_r[256], s_s[256], s_off[256];
    for (int j = threadIdx.x; j < cols; j += blockDim.x) {
        if (j < p.kk) { const int c = j % p.C, rs = j / p.C, ss = rs % p.ksz, r = rs / p.ksz; s_r[j] = r - p.pad; s_s[j] = ss - p.pad; s_off[j] = ((r - p.pad) * p.W + (ss - p.pad)) * p.C + c; }
        else { s_r[j] = -(1 << 20); s_s[j] = 0; s_off[j] = 0; }   // beyond the taps: never inside the image
    }
    __syncthreads();
    const unsigned short* __restrict__ src16 = reinterpret_cast<const unsigned short*>(src);
    for (long long id = blockIdx.x * (long long)blockDim.x + threadIdx.x; id < total; id += (long long)gridDim.x * blockDim.x) {
        const int g = G == 4 ? (int)(id & 3) : (int)(id % G); const long long row = G == 4 ? id >> 2 : id / G;
        const int q = (int)(row % p.Q); const long long t = row / p.Q; const int pr = (int)(t % p.P); const int n = (int)(t / p.P);
        const int y0 = pr * p.stride, x0 = q * p.stride;
        const long long base = (((long long)n * p.H + y0) * p.W + x0) * p.C;
        unsigned short h[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = g * 8 + e;
            const int y = y0 + s_r[j], xx = x0 + s_s[j];
            const bool in = y >= 0 && y < p.H && xx >= 0 && xx < p.W;
            h[e] = in ? src16[base + s_off[j]] : (unsigned short)0;
        }
        *reinterpret_cast<uint4*>((__nv_bfloat16*)p.dst + row * cols + g * 8) =
            make_uint4(h[0] | ((unsigned)h[1] << 16), h[2] | ((unsigned)h[3] << 16), h[4] | ((unsigned)h[5] << 16), h[6] | ((unsigned)h[7] << 16));
        if (id < (long long)p.K * G) {                             // weights: w[k][kk] -> w32[k][cols]
            const int kx = (int)(id / G);
            __align__(16) __nv_bfloat16 wv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) { const int j = g * 8 + e; wv[e] = j < p.kk ? ((const __nv_bfloat16*)p.w)[(long long)kx * p.kk + j] : __float2bfloat16(0.f); }
            *reinterpret_cast<uint4*>((__nv_bfloat16*)p.w32 + (long long)kx * cols + g * 8) = *reinterpret_cast<const uint4*>(wv);
        }
    }
}
void launch_im2col(const ColProb* d, int nprob, long long max_rows, cudaStream_t s) {
    long long gx = (max_rows * 4 + 255) / 256; if (gx > 148 * 16) gx = 148 * 16; if (gx < 1) gx = 1;
    im2col_kernel<<<dim3((unsigned)gx, nprob), 256, 0, s>>>(d);
}

// dst[r][0..cols) = src[r][0..cols) for rows of different pitch (fp32): the weight gradient of an im2col'ed stem, computed with
// the padded column count, goes to its place in the gradient vector
__global__ void repack_rows_kernel(const ConvProb* __restrict__ probs) {
    const ConvProb& p = probs[blockIdx.y];
    const float* src = (const float*)p.act; float* dst = (float*)p.out;
    const int n = p.M * p.Ncol;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const int r = i / p.Ncol, c = i - r * p.Ncol;
        dst[i] = src[(long long)r * p.Kred + c];
    }
}
void launch_repack_rows(const ConvProb* d, int nprob, int max_elems, cudaStream_t s) {
    repack_rows_kernel<<<dim3(std::max(1, std::min((max_elems + 255) / 256, 148)), nprob), 256, 0, s>>>(d);
}

}  // namespace resist
