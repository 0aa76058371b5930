// Bandwidth kernels over the flat parameter arrays: the fused SGD-momentum update (Algorithm 1, the
// local update W_s = W_s - eta dL/dW_s), the scatter of the global parameters into the S working
// copies (the hand-out step of Algorithm 1), and the reassembly aggregate(.) (Sec. 2.3, Appendix B).
// Work is described by a table of segments (contiguous runs of parameters treated alike); every CTA
// owns one 4096-element chunk of one segment, found by binary search, and moves 16 bytes per thread
// per access when the chunk starts on a 16-byte boundary.
#include "internal.h"

namespace resist {

__device__ __forceinline__ const Segment& find_segment(const Segment* segs, int nseg, long long chunk) {
    int lo = 0, hi = nseg - 1;
    while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (segs[mid].chunk0 <= chunk) lo = mid; else hi = mid - 1; }
    return segs[lo];
}

struct Range { long long base; int len; };
__device__ __forceinline__ Range chunk_range(const Segment& sg, long long chunk) {
    const long long off = (chunk - sg.chunk0) * SEG_CHUNK;
    long long len = sg.len - off; if (len > SEG_CHUNK) len = SEG_CHUNK;
    return Range{sg.begin + off, (int)len};
}

__device__ __forceinline__ unsigned pack_bf16x2(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<unsigned*>(&h);
}

// v = mu*v + (g + wd*w);  w = w - lr*v;  bf16 copy of w refreshed for the convolutions
template <bool SHADOW>
__global__ void __launch_bounds__(256) sgd_kernel(const Segment* __restrict__ segs, int nseg, ParamArrays pa,
                                                  float lr, float mu, float wd) {
    const Segment& sg = find_segment(segs, nseg, blockIdx.x);
    const Range r = chunk_range(sg, blockIdx.x);
    const long long o = (long long)sg.sub * pa.n + r.base;
    float* __restrict__ w = pa.w + o; float* __restrict__ v = pa.v + o; const float* __restrict__ g = pa.g + o;
    __nv_bfloat16* __restrict__ wb = pa.wb + o;
    int done = 0;
    if ((o & 3) == 0) {
        const int nq = r.len >> 2;
        for (int q = threadIdx.x; q < nq; q += 256) {
            float4 gg = reinterpret_cast<const float4*>(g)[q], vv = reinterpret_cast<float4*>(v)[q], ww = reinterpret_cast<float4*>(w)[q];
            vv.x = fmaf(mu, vv.x, fmaf(wd, ww.x, gg.x)); ww.x = fmaf(-lr, vv.x, ww.x);
            vv.y = fmaf(mu, vv.y, fmaf(wd, ww.y, gg.y)); ww.y = fmaf(-lr, vv.y, ww.y);
            vv.z = fmaf(mu, vv.z, fmaf(wd, ww.z, gg.z)); ww.z = fmaf(-lr, vv.z, ww.z);
            vv.w = fmaf(mu, vv.w, fmaf(wd, ww.w, gg.w)); ww.w = fmaf(-lr, vv.w, ww.w);
            reinterpret_cast<float4*>(v)[q] = vv; reinterpret_cast<float4*>(w)[q] = ww;
            if (SHADOW) reinterpret_cast<uint2*>(wb)[q] = make_uint2(pack_bf16x2(ww.x, ww.y), pack_bf16x2(ww.z, ww.w));
        }
        done = nq << 2;
    }
    for (int i = done + threadIdx.x; i < r.len; i += 256) {
        float vv = fmaf(mu, v[i], fmaf(wd, w[i], g[i])); float ww = fmaf(-lr, vv, w[i]);
        v[i] = vv; w[i] = ww; if (SHADOW) wb[i] = __float2bfloat16_rn(ww);
    }
}

// working copy <- global; momentum <- 0 (restart); bf16 copy <- round(global)
template <bool SHADOW, bool ZERO_V>
__global__ void __launch_bounds__(256) scatter_kernel(const Segment* __restrict__ segs, int nseg, ParamArrays pa) {
    const Segment& sg = find_segment(segs, nseg, blockIdx.x);
    const Range r = chunk_range(sg, blockIdx.x);
    const long long o = (long long)sg.sub * pa.n + r.base;
    const float* __restrict__ src = pa.global + r.base;
    float* __restrict__ w = pa.w + o; float* __restrict__ v = pa.v + o; __nv_bfloat16* __restrict__ wb = pa.wb + o;
    int done = 0;
    if (((o | r.base) & 3) == 0) {
        const int nq = r.len >> 2;
        for (int q = threadIdx.x; q < nq; q += 256) {
            float4 x = reinterpret_cast<const float4*>(src)[q];
            reinterpret_cast<float4*>(w)[q] = x;
            if (ZERO_V) reinterpret_cast<float4*>(v)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (SHADOW) reinterpret_cast<uint2*>(wb)[q] = make_uint2(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w));
        }
        done = nq << 2;
    }
    for (int i = done + threadIdx.x; i < r.len; i += 256) {
        float x = src[i]; w[i] = x; if (ZERO_V) v[i] = 0.f; if (SHADOW) wb[i] = __float2bfloat16_rn(x);
    }
}

__global__ void __launch_bounds__(256) scatter_buffers_kernel(const Segment* __restrict__ segs, int nseg, ParamArrays pa) {
    const Segment& sg = find_segment(segs, nseg, blockIdx.x);
    const Range r = chunk_range(sg, blockIdx.x);
    const float* __restrict__ src = pa.global_buf + r.base;
    float* __restrict__ dst = pa.buf + (long long)sg.sub * pa.nbuf + r.base;
    for (int i = threadIdx.x; i < r.len; i += 256) dst[i] = src[i];
}

// global <- first + (sum over the other owners of (w_s - first)) / count, owners ascending; one owner: copy.
// Explicit round-to-nearest intrinsics keep the compiler from contracting the arithmetic.
__device__ __forceinline__ float mean_of_owners(const float* __restrict__ sub, long long stride, long long i,
                                                unsigned mask, int S, float keep) {
    int cnt = 0; float first = 0.f, acc = 0.f;
    for (int s = 0; s < S; ++s)
        if (mask >> s & 1u) {
            const float x = sub[(long long)s * stride + i];
            if (cnt == 0) first = x; else acc = __fadd_rn(acc, __fsub_rn(x, first));
            ++cnt;
        }
    if (cnt == 0) return keep;
    if (cnt == 1) return first;
    return __fadd_rn(first, __fdiv_rn(acc, (float)cnt));
}

// Segment::sub selects the array pair: 0 = parameters, 1 = BN running statistics (one launch serves both).
__device__ __forceinline__ void acc_diff(float4& acc, const float4& x, const float4& first) {
    acc.x = __fadd_rn(acc.x, __fsub_rn(x.x, first.x)); acc.y = __fadd_rn(acc.y, __fsub_rn(x.y, first.y));
    acc.z = __fadd_rn(acc.z, __fsub_rn(x.z, first.z)); acc.w = __fadd_rn(acc.w, __fsub_rn(x.w, first.w));
}
__global__ void __launch_bounds__(256, 3) aggregate_kernel(const Segment* __restrict__ segs, int nseg, AggArrays arr, int S) {
    const Segment& sg = find_segment(segs, nseg, blockIdx.x);
    const long long off = ((long long)blockIdx.x - sg.chunk0) * AGG_CHUNK;
    long long rem = sg.len - off; if (rem > AGG_CHUNK) rem = AGG_CHUNK;
    const Range r{sg.begin + off, (int)rem};
    const int which = sg.sub != 0;
    const float* __restrict__ sub = which ? arr.sub_b : arr.sub_p; const long long stride = which ? arr.stride_b : arr.stride_p;
    float* __restrict__ global = which ? arr.global_b : arr.global_p;
    const unsigned mask = sg.mask & (S >= 32 ? 0xffffffffu : ((1u << S) - 1u));   // owners are sub-ResNets 0 .. S-1
    int done = 0;
    if (((r.base | stride) & 3) == 0) {
        const int nq = r.len >> 2;
        const int cnt = __popc(mask);
        // The kernel is bound by the bytes it keeps in flight: four 16-byte groups per thread at a time, and the loads of TWO
        // owners (ascending; the mask is the segment's, so the loop is uniform over the CTA) in flight together.  The arithmetic per element is the scalar
        // routine's, in its order: first + (sum over the other owners of (w_s - first)) / count.
        if (cnt >= 1) {
            for (int q0 = threadIdx.x; q0 < nq; q0 += 4 * 256) {
                float4 first[4], acc[4];
                unsigned m = mask;
                const int s0 = __ffs(m) - 1; m &= m - 1;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int q = q0 + u * 256;
                    first[u] = q < nq ? *reinterpret_cast<const float4*>(sub + (long long)s0 * stride + r.base + 4LL * q) : make_float4(0.f, 0.f, 0.f, 0.f);
                    acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                while (m) {
                    const int sa = __ffs(m) - 1; m &= m - 1;
                    const int sb = m ? __ffs(m) - 1 : -1; if (m) m &= m - 1;
                    float4 xa[4], xb[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int q = q0 + u * 256;
                        xa[u] = q < nq ? *reinterpret_cast<const float4*>(sub + (long long)sa * stride + r.base + 4LL * q) : first[u];
                        xb[u] = (sb >= 0 && q < nq) ? *reinterpret_cast<const float4*>(sub + (long long)sb * stride + r.base + 4LL * q) : first[u];
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) acc_diff(acc[u], xa[u], first[u]);
                    if (sb >= 0) {
#pragma unroll
                        for (int u = 0; u < 4; ++u) acc_diff(acc[u], xb[u], first[u]);
                    }
                }
                const float c = (float)cnt;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int q = q0 + u * 256;
                    if (q >= nq) continue;
                    float4 out = first[u];
                    if (cnt > 1) {
                    out.x = __fadd_rn(first[u].x, __fdiv_rn(acc[u].x, c)); out.y = __fadd_rn(first[u].y, __fdiv_rn(acc[u].y, c));
                    out.z = __fadd_rn(first[u].z, __fdiv_rn(acc[u].z, c)); out.w = __fadd_rn(first[u].w, __fdiv_rn(acc[u].w, c));
                    }
                    *reinterpret_cast<float4*>(global + r.base + 4LL * q) = out;
                }
            }
        }
        done = nq << 2;
    }
    for (int k = done + threadIdx.x; k < r.len; k += 256) {
        const long long i = r.base + k;
        global[i] = mean_of_owners(sub, stride, i, mask, S, global[i]);
    }
}

void launch_sgd(const Segment* d, int nseg, long long nchunks, ParamArrays pa, float lr, float mu, float wd,
                bool shadow, cudaStream_t s) {
    if (nchunks <= 0) return;
    if (shadow) sgd_kernel<true><<<(unsigned)nchunks, 256, 0, s>>>(d, nseg, pa, lr, mu, wd);
    else sgd_kernel<false><<<(unsigned)nchunks, 256, 0, s>>>(d, nseg, pa, lr, mu, wd);
}
void launch_scatter(const Segment* d, int nseg, long long nchunks, ParamArrays pa, bool zero_momentum, bool shadow,
                    cudaStream_t s) {
    if (nchunks <= 0) return;
    const unsigned g = (unsigned)nchunks;
    if (shadow) { if (zero_momentum) scatter_kernel<true, true><<<g, 256, 0, s>>>(d, nseg, pa);
                  else scatter_kernel<true, false><<<g, 256, 0, s>>>(d, nseg, pa); }
    else { if (zero_momentum) scatter_kernel<false, true><<<g, 256, 0, s>>>(d, nseg, pa);
           else scatter_kernel<false, false><<<g, 256, 0, s>>>(d, nseg, pa); }
}
void launch_scatter_buffers(const Segment* d, int nseg, long long nchunks, ParamArrays pa, cudaStream_t s) {
    if (nchunks <= 0) return;
    scatter_buffers_kernel<<<(unsigned)nchunks, 256, 0, s>>>(d, nseg, pa);
}
void launch_aggregate(const Segment* d, int nseg, long long nchunks, const AggArrays& arr, int S, cudaStream_t s) {
    if (nchunks <= 0) return;
    aggregate_kernel<<<(unsigned)nchunks, 256, 0, s>>>(d, nseg, arr, S);
}

}  // namespace resist
