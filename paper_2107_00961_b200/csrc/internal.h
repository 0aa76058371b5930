// Internal declarations shared by the runtime and the kernel files of the ResIST library.
// Every kernel is a "grouped" kernel: it receives a device array of problem descriptors and
// blockIdx.y selects the problem, so the S sub-ResNets of one layer slot run in one launch.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace resist {

enum ConvMode { CONV_FWD = 0, CONV_DGRAD = 1, CONV_WGRAD = 2 };

// One convolution problem, any mode.  Geometry always describes the FORWARD convolution:
// input [N,H,W,C], weights [K,ksz,ksz,C], output [N,P,Q,K].
struct ConvProb {
    const void* act;      // fwd: input a;      dgrad: dy;            wgrad: input a
    const void* wgt;      // fwd: weights;      dgrad: weights;       wgrad: dy
    const void* add;      // optional tensor added to the result (shape of out), or nullptr
    void* out;            // fwd: y (T);        dgrad: da (T);        wgrad: dw (fp32, [K][ksz][ksz][C])
    float* partial;       // wgrad split-K workspace [splits][K*ksz*ksz*C], or nullptr
    int N, H, W, C, K, ksz, stride, pad, P, Q;
    int M, Ncol, Kred;    // GEMM extents of this mode
    int tiles_m, tiles_n, splits, ktiles_per_split;
    float scale;          // result = scale*acc + add
    int wg_ld, wg_cols;   // wgrad of a 1x1 problem on an im2col'ed input: row stride and valid columns of dw (0: K x C dense)
    int dy_sub;           // backward of a stride-2 layer as a stride-1 problem: 2 = dy is stored compact [N,dy_P,dy_Q,K] and read as if
    int dy_P, dy_Q;       //   zero-stuffed to H x W (only even positions exist); 0 or 1 = dy is stored at the problem's resolution
    int out_compact;      // dgrad of a stride-2 1x1 layer on tcgen05: out is [N,P,Q,C], the gradient at the even input positions (all others are zero)
    int add_sub;          // 2: `add` is such a compact tensor [N,(H+1)/2,(W+1)/2,Ncol] and is added at the even positions of the H x W result only
    float* stat_tiles;    // forward on tcgen05: per 128-position tile, the column sums and sums of squares of the stored output [tiles][2][K], or nullptr
};

// One batch-normalisation + ReLU problem over x [m, C] (forward or backward).
struct BnProb {
    const void* x;        // pre-normalisation tensor (T)
    void* a;              // forward output relu(bn(x)) (T)
    const void* da;       // backward: gradient w.r.t. a (T)
    void* dx;             // backward: gradient w.r.t. x (T)
    const void* add;      // backward: tensor added to dx (skip-path gradient), or nullptr
    const float* gamma; const float* beta;
    float* dgamma; float* dbeta;
    float* run_mean; float* run_var;   // forward: updated when non-null
    double* partial;      // [chunks][2][C]
    float* stat;          // [4][C]: mean, invstd, sum dz, sum dz*xhat
    long long m;
    int C, chunks, rows_per_chunk;
    float eps, momentum;
    int eval;             // 1: use running statistics (no batch statistics)
    int vec;              // 1: bf16 fast path (16-byte accesses, 8 channels per thread)
};

// How the rows of a BN problem are cut into chunks (one CTA each) and whether the vector path applies.
inline void bn_chunking(BnProb& p, bool bf16, int target_chunks = 0) {
    const int C = p.C; const long long m = p.m;
    const int G = C / 8;
    const bool pow2 = G > 0 && (G & (G - 1)) == 0;
    const bool aligned = ((((uintptr_t)p.x) | ((uintptr_t)p.a) | ((uintptr_t)p.da) | ((uintptr_t)p.dx) | ((uintptr_t)p.add) |
                            ((uintptr_t)p.gamma) | ((uintptr_t)p.beta) | ((uintptr_t)p.stat)) & 15) == 0;
    p.vec = (bf16 && C % 8 == 0 && pow2 && G <= 256 && aligned) ? 1 : 0;
    long long rpc;
    if (p.vec) { const int R = 256 / G; rpc = (long long)R * 16; }
    else { const int nl = C < 256 ? C : 256, R = 256 / nl; rpc = (long long)R * 32; }
    const long long lim = (m + 1023) / 1024; if (rpc < lim) rpc = lim;
    if (p.vec && target_chunks > 0 && (m + rpc - 1) / rpc < target_chunks) {      // more, smaller chunks (whole sweeps of the CTA's rows)
        const int R = 256 / G;
        rpc = ((m + target_chunks - 1) / target_chunks + R - 1) / R * R;
        if (rpc < 32 * R) rpc = 32 * R;            // every CTA of the cooperative kernels re-adds all chunks' sums: few chunks for small problems
    }
    p.rows_per_chunk = (int)rpc; p.chunks = (int)((m + rpc - 1) / rpc);
}

// im2col of a few-channel input: dst [N*P*Q][cols] (bf16, columns (r, s, c), zero beyond C*ksz*ksz), and the
// layer's weights packed alike: w32 [K][cols].
struct ColProb {
    const void* src; void* dst; const void* w; void* w32;
    int N, H, W, C, ksz, stride, pad, P, Q, K, kk, cols;   // kk = C*ksz*ksz real columns; cols = row pitch (multiple of 8, <= 256)
};

struct UpProb {           // zero stuffing of a stride-2 layer's dy: src [N,P,Q,K] -> dst [N,H,W,K] (bf16, K % 8 == 0)
    const void* src; void* dst; int N, H, W, K, P, Q;
};

struct PoolProb {         // 3x3 stride-2 max-pool, pad 1: x [N,H,W,C] -> y [N,P,Q,C]
    const void* x; void* y; int* arg; const void* dy; void* dx;
    int N, H, W, C, P, Q;
};

struct HeadProb {         // global average pool + linear head + mean softmax cross-entropy
    const void* a;        // final activation (T) [B, HW, C]
    void* da;             // its gradient (T)
    const float* w; const float* b; float* dw; float* db;
    float* pooled;        // [B, C]
    float* dpooled;       // [B, C]
    float* logits;        // [B, classes]
    float* dlogits;       // [B, classes]
    const int* labels;
    float* loss;          // [1]
    float* loss_user;     // optional copy for the caller
    int* correct;         // optional top-1 count
    float* logits_user;   // optional copy for the caller
    int B, HW, C, classes;
};

// A contiguous run of parameters treated alike by the bandwidth kernels.
struct Segment {
    long long begin;      // offset in the flat vector
    long long len;
    long long chunk0;     // first chunk index of this segment in the launch
    unsigned mask;        // aggregate: owners; scatter/sgd: unused
    int sub;              // scatter/sgd: sub-ResNet index
};

struct ParamArrays {      // device pointers of the flat arrays
    float* global; float* global_buf;
    float* w;  float* v;  float* g;  __nv_bfloat16* wb;  float* buf;   // [S][n] each (buf: [S][n_buffers])
    long long n, nbuf;
};

constexpr int SEG_CHUNK = 4096;   // elements per CTA in the segment kernels
constexpr int AGG_CHUNK = 8192;   // elements per CTA of the aggregate kernel (two rounds of four 16-byte groups per thread)

// ---- launchers (kernels_ref.cu)
void launch_conv_ref(const ConvProb* d, int nprob, int max_tiles, int mode, bool bf16, cudaStream_t s);
void launch_splitk_reduce(const ConvProb* d, int nprob, int max_elems, cudaStream_t s);
void launch_bn_stats(const BnProb* d, int nprob, int max_chunks, int max_c, bool bf16, cudaStream_t s);
void launch_bn_apply(const BnProb* d, int nprob, long long max_elems, bool bf16, cudaStream_t s);
void launch_bn_bwd_reduce(const BnProb* d, int nprob, int max_chunks, int max_c, bool bf16, cudaStream_t s);
void launch_bn_bwd_apply(const BnProb* d, int nprob, long long max_elems, bool bf16, cudaStream_t s);
void launch_maxpool_fwd(const PoolProb* d, int nprob, long long max_elems, bool bf16, cudaStream_t s);
void launch_maxpool_bwd(const PoolProb* d, int nprob, long long max_elems, bool bf16, cudaStream_t s);
void launch_head_fwd(const HeadProb* d, int nprob, int maxB, int maxC, int max_classes, bool bf16, cudaStream_t s);
void launch_head_bwd(const HeadProb* d, int nprob, int maxB, int maxC, int max_classes, long long max_elems,
                     bool bf16, cudaStream_t s);

// statistics, finalisation and apply of BN+ReLU in one cooperative launch (bf16 vector path, training mode); false if the grid cannot be co-resident
bool launch_bn_fused(const BnProb* d, int nprob, int max_chunks, int backward, cudaStream_t s);   // kernels_ref.cu
void launch_im2col(const ColProb* d, int nprob, long long max_rows, cudaStream_t s);      // kernels_ref.cu
void launch_repack_rows(const ConvProb* d, int nprob, int max_elems, cudaStream_t s);     // kernels_ref.cu
void launch_zero_stuff(const UpProb* d, int nprob, long long max_vecs, cudaStream_t s);   // conv_tc.cu

// ---- launchers (kernels_bw.cu)
void launch_sgd(const Segment* d, int nseg, long long nchunks, ParamArrays pa, float lr, float mu, float wd,
                bool shadow, cudaStream_t s);
void launch_scatter(const Segment* d, int nseg, long long nchunks, ParamArrays pa, bool zero_momentum, bool shadow,
                    cudaStream_t s);
void launch_scatter_buffers(const Segment* d, int nseg, long long nchunks, ParamArrays pa, cudaStream_t s);
struct AggArrays { const float* sub_p; const float* sub_b; long long stride_p, stride_b; float* global_p; float* global_b; };   // _p parameters, _b BN running statistics
void launch_aggregate(const Segment* d, int nseg, long long nchunks, const AggArrays& arr, int S, cudaStream_t s);

}  // namespace resist
