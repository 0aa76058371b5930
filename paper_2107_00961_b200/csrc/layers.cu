// Layer-level entry points: one convolution (forward, dgrad or wgrad) or one BN+ReLU (forward, backward)
// on caller-owned device tensors, run by the same kernels the local step uses.
#include <algorithm>
#include <string>
#include <vector>
#include "runtime.h"

namespace resist {
bool conv_tc_supported(const ConvProb& p, int mode);
int conv_tc_fill(const ConvProb& p, int mode, void* host_tc);
int conv_tc_count(const ConvProb& p, int mode);
size_t conv_tc_merge(size_t a, size_t b);
size_t conv_tc_prob_bytes();
int conv_tc_tiles(const void* host_tc);
size_t conv_tc_smem(const void* host_tc);
void launch_conv_tc_probs(const void* d_tc, int nprob, int max_tiles, size_t max_smem, cudaStream_t s);
int conv_tc_read_status();
bool conv_wgrad_tc_supported(const ConvProb& p, int target_ctas, size_t* partial_bytes);
bool conv_wgrad_tc_fill(const ConvProb& p, int target_ctas, void* host_tc);
size_t conv_wgrad_tc_prob_bytes();
int conv_wgrad_tc_ctas(const void* h);
size_t conv_wgrad_tc_smem(const void* h);
long long conv_wgrad_tc_out_elems(const void* h);
void launch_conv_wgrad_tc_probs(const void* d_tc, int nprob, int max_ctas, size_t max_smem, long long max_out, cudaStream_t s);
bool conv_mma_supported(const ConvProb& p, int mode);
bool conv_mma_fill(const ConvProb& p, int mode, void* host, const BnProb* bn = nullptr);
size_t conv_mma_prob_bytes();
int conv_mma_tiles(const void* h);
size_t conv_mma_smem(const void* h);
bool launch_conv_mma_probs(const void* d, int nprob, int max_tiles, size_t max_smem, int variant, cudaStream_t s, bool pdl = false);
int conv_mma_pick_variant(const ConvProb& p, int mode);
bool conv_wgrad_mma_supported(const ConvProb& p, int target_ctas, size_t* partial_bytes);
bool conv_wgrad_mma_fill(const ConvProb& p, int target_ctas, void* host);
size_t conv_wgrad_mma_prob_bytes();
int conv_wgrad_mma_ctas(const void* h);
size_t conv_wgrad_mma_smem(const void* h);
long long conv_wgrad_mma_out_elems(const void* h);
void launch_conv_wgrad_mma_probs(const void* d, int nprob, int max_ctas, size_t max_smem, long long max_out, int variant, cudaStream_t s, bool pdl = false);
int conv_wgrad_mma_pick_variant(const ConvProb& p, int target_ctas);
}
using namespace resist;

static thread_local std::string g_layer_error;
extern "C" const char* resist_layer_last_error(void) { return g_layer_error.c_str(); }

static int out_dim(int h, int k, int stride) { return (h + 2 * ((k - 1) / 2) - k) / stride + 1; }

extern "C" int resist_conv2d(int32_t mode, int32_t dtype, int32_t backend, const void* act, const void* wgt, const void* add,
                             void* out, int32_t N, int32_t H, int32_t W, int32_t C, int32_t K, int32_t ksz, int32_t stride,
                             float scale, int32_t* used_backend, resist_stream stream) {
    if (!act || !wgt || !out || N < 1 || H < 1 || W < 1 || C < 1 || K < 1 || ksz < 1 || ksz % 2 == 0 || stride < 1 || mode < 0 || mode > 2) {
        g_layer_error = "bad argument"; return RESIST_EINVAL; }
    if (dtype != RESIST_F32 && dtype != RESIST_BF16) { g_layer_error = "bad dtype"; return RESIST_EINVAL; }
    cudaStream_t st = (cudaStream_t)stream;
    ConvProb p{};
    p.N = N; p.H = H; p.W = W; p.C = C; p.K = K; p.ksz = ksz; p.stride = stride; p.pad = (ksz - 1) / 2;
    p.P = out_dim(H, ksz, stride); p.Q = out_dim(W, ksz, stride); p.scale = scale; p.add = add; p.out = out;
    p.act = act; p.wgt = wgt;
    const long long rows_out = (long long)N * p.P * p.Q, rows_in = (long long)N * H * W;
    if (mode == CONV_FWD) { p.M = (int)rows_out; p.Ncol = K; p.Kred = ksz * ksz * C; }
    else if (mode == CONV_DGRAD) { p.M = (int)rows_in; p.Ncol = C; p.Kred = ksz * ksz * K; }
    else { p.M = K; p.Ncol = ksz * ksz * C; p.Kred = (int)rows_out; p.add = nullptr; }
    p.tiles_m = (p.M + 63) / 64; p.tiles_n = (p.Ncol + 63) / 64; p.splits = 1;
    const int ktiles = (p.Kred + 15) / 16; p.ktiles_per_split = ktiles;
    int sm = 148; int dev = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
    // which kernel family: 0 CUDA cores, 1 tcgen05, 2 warp-level MMA
    auto pick = [&](const ConvProb& q, size_t* pb) -> int {
        if (dtype != RESIST_BF16 || backend == RESIST_CONV_CUDA_CORES) return 0;
        const bool want_mma = backend == RESIST_CONV_AUTO || backend == RESIST_CONV_WARP_MMA;
        const bool want_tc = backend == RESIST_CONV_AUTO || backend == RESIST_CONV_TCGEN05;
        if (mode == CONV_WGRAD) {
            if (want_mma && conv_wgrad_mma_supported(q, 2 * sm, pb)) return 2;
            if (want_tc && conv_wgrad_tc_supported(q, 2 * sm, pb)) return 1;
            return 0;
        }
        if (want_mma && conv_mma_supported(q, mode)) return 2;
        if (want_tc && conv_tc_supported(q, mode)) return 1;
        return 0;
    };
    // backward of a stride-2 layer on the warp-MMA kernels: stride-1 problem on a zero-stuffed dy (the tcgen05 kernels take the
    // stride-2 problem as it is)
    char* up = nullptr;
    if (stride == 2 && mode != CONV_FWD && K % 8 == 0) {
        ConvProb q = p; q.stride = 1; q.P = H; q.Q = W;
        if (mode == CONV_DGRAD) q.M = (int)rows_in; else q.Kred = (int)rows_in;
        size_t pb = 0;
        if (pick(q, &pb) == 2) {
            if (cudaMalloc(&up, (size_t)N * H * W * K * 2 + 256) != cudaSuccess) { g_layer_error = "cudaMalloc failed"; return RESIST_ENOMEM; }
            UpProb u{mode == CONV_DGRAD ? p.act : p.wgt, up + 256, N, H, W, K, p.P, p.Q};
            cudaMemcpyAsync(up, &u, sizeof(u), cudaMemcpyHostToDevice, st);
            launch_zero_stuff((const UpProb*)up, 1, (long long)N * H * W * (K / 8), st);
            if (mode == CONV_DGRAD) q.act = up + 256; else q.wgt = up + 256;
            p = q;
        }
    }
    size_t wg_partial = 0;
    const int be = pick(p, &wg_partial);
    if (used_backend) *used_backend = be;
    size_t scratch = 0;
    std::vector<char> hd;                                      // host copy of the kernel family's own descriptor
    int n_tc = 1;
    if (be == 1) { n_tc = mode == CONV_WGRAD ? 1 : conv_tc_count(p, mode); hd.resize(mode == CONV_WGRAD ? conv_wgrad_tc_prob_bytes() : (size_t)n_tc * conv_tc_prob_bytes()); }
    if (be == 2) hd.resize(mode == CONV_WGRAD ? conv_wgrad_mma_prob_bytes() : conv_mma_prob_bytes());
    const size_t hd_room = (hd.size() + 255) / 256 * 256;
    if (be && mode == CONV_WGRAD) scratch = hd_room + wg_partial; else if (be) scratch = hd_room;
    if (!be && mode == CONV_WGRAD) {
        const int tiles = p.tiles_m * p.tiles_n;
        int want = (2 * sm + tiles - 1) / tiles; want = std::max(1, std::min(std::min(want, 64), ktiles));
        p.ktiles_per_split = (ktiles + want - 1) / want; p.splits = (ktiles + p.ktiles_per_split - 1) / p.ktiles_per_split;
        if (p.splits > 1) scratch = (size_t)p.splits * p.M * p.Ncol * 4;
    }
    char* blob = nullptr;
    cudaError_t e = cudaMalloc(&blob, 1024 + scratch);
    if (e != cudaSuccess) { cudaFree(up); g_layer_error = cudaGetErrorString(e); return RESIST_ENOMEM; }
    if (!be && p.splits > 1) p.partial = (float*)(blob + 1024);
    if (be && mode == CONV_WGRAD) p.partial = (float*)(blob + 1024 + hd_room);
    bool filled = true;
    if (be == 1) filled = mode == CONV_WGRAD ? conv_wgrad_tc_fill(p, 2 * sm, hd.data()) : conv_tc_fill(p, mode, hd.data()) == n_tc;
    // dgrad of a stride-2 1x1 layer on tcgen05 stores the even positions only: the rest of the gradient is zero
    // (with a residual the rest is the residual itself)
    if (be == 1 && mode == CONV_DGRAD && ksz == 1 && stride == 2) {
        if (add) cudaMemcpyAsync(out, add, (size_t)rows_in * C * 2, cudaMemcpyDeviceToDevice, st);
        else cudaMemsetAsync(out, 0, (size_t)rows_in * C * 2, st);
    }
    if (be == 2) filled = mode == CONV_WGRAD ? conv_wgrad_mma_fill(p, 2 * sm, hd.data()) : conv_mma_fill(p, mode, hd.data());
    if (!filled) { cudaFree(blob); cudaFree(up); g_layer_error = "descriptor set-up failed"; return RESIST_ECUDA; }
    e = cudaMemcpyAsync(blob, &p, sizeof(p), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && be) e = cudaMemcpyAsync(blob + 1024, hd.data(), hd.size(), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) {
        if (be == 1 && mode == CONV_WGRAD) launch_conv_wgrad_tc_probs(blob + 1024, 1, conv_wgrad_tc_ctas(hd.data()), conv_wgrad_tc_smem(hd.data()), conv_wgrad_tc_out_elems(hd.data()), st);
        else if (be == 1) {
            int tiles = 0; size_t packed = 0;
            for (int i = 0; i < n_tc; ++i) { const char* h = hd.data() + (size_t)i * conv_tc_prob_bytes(); tiles = std::max(tiles, conv_tc_tiles(h)); packed = conv_tc_merge(packed, conv_tc_smem(h)); }
            launch_conv_tc_probs(blob + 1024, n_tc, tiles, packed, st);
        }
        else if (be == 2 && mode == CONV_WGRAD) launch_conv_wgrad_mma_probs(blob + 1024, 1, conv_wgrad_mma_ctas(hd.data()), conv_wgrad_mma_smem(hd.data()), conv_wgrad_mma_out_elems(hd.data()), conv_wgrad_mma_pick_variant(p, 2 * sm), st);
        else if (be == 2) launch_conv_mma_probs(blob + 1024, 1, conv_mma_tiles(hd.data()), conv_mma_smem(hd.data()), conv_mma_pick_variant(p, mode), st);
        else {
            launch_conv_ref((ConvProb*)blob, 1, p.tiles_m * p.tiles_n * p.splits, mode, dtype == RESIST_BF16, st);
            if (mode == CONV_WGRAD && p.splits > 1) launch_splitk_reduce((ConvProb*)blob, 1, p.M * p.Ncol, st);
        }
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(blob); cudaFree(up);
    if (e != cudaSuccess) { g_layer_error = cudaGetErrorString(e); return RESIST_ECUDA; }
    if (be == 1) { const int stv = conv_tc_read_status();
        if (stv) { g_layer_error = "a bounded device-side wait gave up (code " + std::to_string(stv) + ")"; return RESIST_ETIMEOUT; } }
    return RESIST_OK;
}

static void fill_bn(BnProb& p, int64_t m, int C, bool bf16) {
    p.m = m; p.C = C;
    bn_chunking(p, bf16);
}

extern "C" int resist_bn_relu_forward(int32_t dtype, const void* x, const float* gamma, const float* beta, void* a, float* stat,
                                      float* run_mean, float* run_var, int64_t m, int32_t C, float eps, float momentum,
                                      resist_stream stream) {
    if (!x || !gamma || !beta || !a || !stat || m < 1 || C < 1) { g_layer_error = "bad argument"; return RESIST_EINVAL; }
    cudaStream_t st = (cudaStream_t)stream;
    BnProb p{}; p.x = x; p.a = a; p.gamma = gamma; p.beta = beta; p.run_mean = run_mean; p.run_var = run_var; p.stat = stat;
    p.eps = eps; p.momentum = momentum; fill_bn(p, m, C, dtype == RESIST_BF16);
    char* blob = nullptr;
    cudaError_t e = cudaMalloc(&blob, 1024 + (size_t)p.chunks * 2 * C * 8);
    if (e != cudaSuccess) { g_layer_error = cudaGetErrorString(e); return RESIST_ENOMEM; }
    p.partial = (double*)(blob + 1024);
    e = cudaMemcpyAsync(blob, &p, sizeof(p), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) {
        launch_bn_stats((BnProb*)blob, 1, p.chunks, C, dtype == RESIST_BF16, st);
        launch_bn_apply((BnProb*)blob, 1, m * C, dtype == RESIST_BF16, st);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(blob);
    if (e != cudaSuccess) { g_layer_error = cudaGetErrorString(e); return RESIST_ECUDA; }
    return RESIST_OK;
}

extern "C" int resist_bn_relu_backward(int32_t dtype, const void* x, const void* da, const float* gamma, const float* beta,
                                       float* stat, const void* add, void* dx, float* dgamma, float* dbeta, int64_t m, int32_t C,
                                       resist_stream stream) {
    if (!x || !da || !gamma || !beta || !stat || !dx || !dgamma || !dbeta || m < 1 || C < 1) { g_layer_error = "bad argument"; return RESIST_EINVAL; }
    cudaStream_t st = (cudaStream_t)stream;
    BnProb p{}; p.x = x; p.da = da; p.dx = dx; p.add = add; p.gamma = gamma; p.beta = beta; p.dgamma = dgamma; p.dbeta = dbeta; p.stat = stat;
    fill_bn(p, m, C, dtype == RESIST_BF16);
    char* blob = nullptr;
    cudaError_t e = cudaMalloc(&blob, 1024 + (size_t)p.chunks * 2 * C * 8);
    if (e != cudaSuccess) { g_layer_error = cudaGetErrorString(e); return RESIST_ENOMEM; }
    p.partial = (double*)(blob + 1024);
    e = cudaMemcpyAsync(blob, &p, sizeof(p), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) {
        launch_bn_bwd_reduce((BnProb*)blob, 1, p.chunks, C, dtype == RESIST_BF16, st);
        launch_bn_bwd_apply((BnProb*)blob, 1, m * C, dtype == RESIST_BF16, st);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(blob);
    if (e != cudaSuccess) { g_layer_error = cudaGetErrorString(e); return RESIST_ECUDA; }
    return RESIST_OK;
}

namespace resist {
bool conv_mma_can_fuse_bn(const ConvProb& p, int mode, int C);
size_t conv_mma_bn_partial_bytes(int C, int sms);
int conv_tc_stat_tiles(const ConvProb& p);
void launch_bn_finalize_tiles(const BnProb* d, int nprob, int max_c, cudaStream_t s);
}

// A convolution together with the BN+ReLU that consumes its output, launched the way the local step launches the pair (bf16):
//   mode 0: y = scale * conv(a, w) + add;  a_out = relu(bn(y)) with batch statistics (stat, running statistics updated)
//   mode 1: da = conv^T(dy, w) + add;      dx = BN+ReLU backward of the BN with input x and output gradient da (+ bn_add), dgamma, dbeta
// Warp-MMA family (narrow layers): the BN runs inside the convolution's launch.  tcgen05 family: forward statistics come from the
// per-tile sums of the convolution's epilogue (a finalize launch, then the elementwise pass); backward is the cooperative BN launch
// behind the dgrad.  *used_backend: 1 tcgen05, 2 warp-level MMA.
extern "C" int resist_conv2d_bn_relu(int32_t mode, int32_t backend, const void* act, const void* wgt, const void* add, void* out,
                                     int32_t N, int32_t H, int32_t W, int32_t C, int32_t K, int32_t ksz, int32_t stride, float scale,
                                     const void* x, const float* gamma, const float* beta, float* stat, float* run_mean, float* run_var,
                                     const void* bn_add, void* bn_out, float* dgamma, float* dbeta, float eps, float momentum,
                                     int32_t* used_backend, resist_stream stream) {
    if (!act || !wgt || !out || !gamma || !beta || !stat || !bn_out || mode < 0 || mode > 1 || N < 1 || H < 1 || W < 1 || C < 1 || K < 1 ||
        (ksz != 1 && ksz != 3) || stride < 1 || stride > 2) { g_layer_error = "bad argument"; return RESIST_EINVAL; }
    if (mode == 1 && (!x || !dgamma || !dbeta)) { g_layer_error = "backward needs x, dgamma, dbeta"; return RESIST_EINVAL; }
    cudaStream_t st = (cudaStream_t)stream;
    ConvProb p{};
    p.N = N; p.H = H; p.W = W; p.C = C; p.K = K; p.ksz = ksz; p.stride = stride; p.pad = (ksz - 1) / 2;
    p.P = out_dim(H, ksz, stride); p.Q = out_dim(W, ksz, stride); p.scale = scale; p.add = add; p.out = out; p.act = act; p.wgt = wgt;
    const long long rows_out = (long long)N * p.P * p.Q, rows_in = (long long)N * H * W;
    if (mode == CONV_FWD) { p.M = (int)rows_out; p.Ncol = K; p.Kred = ksz * ksz * C; } else { p.M = (int)rows_in; p.Ncol = C; p.Kred = ksz * ksz * K; }
    int sm = 148; int dev = 0; cudaGetDevice(&dev); cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev);
    BnProb bn{};
    bn.gamma = gamma; bn.beta = beta; bn.stat = stat; bn.run_mean = run_mean; bn.run_var = run_var; bn.eps = eps; bn.momentum = momentum;
    bn.dgamma = dgamma; bn.dbeta = dbeta;
    if (mode == CONV_FWD) { bn.x = out; bn.a = bn_out; bn.m = rows_out; bn.C = K; }
    else { bn.x = x; bn.da = out; bn.dx = bn_out; bn.add = bn_add; bn.m = rows_in; bn.C = C; }
    bn_chunking(bn, true, std::max(8, 2 * sm));
    if (!bn.vec) { g_layer_error = "the BN does not take the bf16 vector path (channels a power of two times 8, 16-byte aligned tensors)"; return RESIST_EUNSUPPORTED; }
    const bool want_mma = backend == RESIST_CONV_AUTO || backend == RESIST_CONV_WARP_MMA, want_tc = backend == RESIST_CONV_AUTO || backend == RESIST_CONV_TCGEN05;
    ConvProb q = p;                                           // the warp-MMA kernels take a stride-2 dgrad as a stride-1 problem that reads dy through its tables
    if (mode == CONV_DGRAD && stride == 2) { q.stride = 1; q.P = H; q.Q = W; q.dy_sub = 2; q.dy_P = p.P; q.dy_Q = p.Q; }
    int be = 0;
    if (want_mma && conv_mma_supported(q, mode) && conv_mma_can_fuse_bn(q, mode, bn.C)) be = 2;
    else if (want_tc && conv_tc_supported(p, mode) && !(mode == CONV_DGRAD && ksz == 1 && stride == 2)) be = 1;
    if (used_backend) *used_backend = be;
    if (!be) { g_layer_error = "no tensor-core family takes this convolution with its BN"; return RESIST_EUNSUPPORTED; }
    const int tiles = be == 1 && mode == CONV_FWD ? conv_tc_stat_tiles(p) : 0;
    const size_t partial_bytes = be == 2 ? conv_mma_bn_partial_bytes(bn.C, sm) : std::max((size_t)bn.chunks * 2 * bn.C * 8, (size_t)tiles * 2 * bn.C * 4);
    const int n_tc = be == 1 ? conv_tc_count(p, mode) : 1;
    std::vector<char> hd(be == 1 ? (size_t)n_tc * conv_tc_prob_bytes() : conv_mma_prob_bytes());
    const size_t hd_room = (hd.size() + 255) / 256 * 256;
    char* blob = nullptr;
    cudaError_t e = cudaMalloc(&blob, 1024 + hd_room + partial_bytes + 256);
    if (e != cudaSuccess) { g_layer_error = cudaGetErrorString(e); return RESIST_ENOMEM; }
    bn.partial = (double*)(blob + 1024 + hd_room);
    bool ok = true;
    if (be == 2) ok = conv_mma_fill(q, mode, hd.data(), &bn);
    else {
        if (mode == CONV_FWD) { p.stat_tiles = (float*)bn.partial; bn.chunks = tiles; }
        ok = conv_tc_fill(p, mode, hd.data()) == n_tc;
    }
    if (!ok) { cudaFree(blob); g_layer_error = "descriptor set-up failed"; return RESIST_ECUDA; }
    e = cudaMemcpyAsync(blob, &bn, sizeof(bn), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(blob + 1024, hd.data(), hd.size(), cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) {
        if (be == 2) {
            if (!launch_conv_mma_probs(blob + 1024, 1, conv_mma_tiles(hd.data()), conv_mma_smem(hd.data()), conv_mma_pick_variant(q, mode) + 512, st)) {
                cudaGetLastError(); cudaFree(blob); g_layer_error = "the fused launch was refused (cooperative grid too large?)"; return RESIST_ECUDA; }
        } else {
            int t = 0; size_t packed = 0;
            for (int i = 0; i < n_tc; ++i) { const char* h = hd.data() + (size_t)i * conv_tc_prob_bytes(); t = std::max(t, conv_tc_tiles(h)); packed = conv_tc_merge(packed, conv_tc_smem(h)); }
            launch_conv_tc_probs(blob + 1024, n_tc, t, packed, st);
            if (mode == CONV_FWD) { launch_bn_finalize_tiles((BnProb*)blob, 1, bn.C, st); launch_bn_apply((BnProb*)blob, 1, bn.m * bn.C, true, st); }
            else if (!(bn.C <= 512 && launch_bn_fused((BnProb*)blob, 1, bn.chunks, 1, st))) {
                cudaGetLastError();
                launch_bn_bwd_reduce((BnProb*)blob, 1, bn.chunks, bn.C, true, st); launch_bn_bwd_apply((BnProb*)blob, 1, bn.m * bn.C, true, st);
            }
        }
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cudaFree(blob);
    if (e != cudaSuccess) { g_layer_error = cudaGetErrorString(e); return RESIST_ECUDA; }
    if (be == 1) { const int stv = conv_tc_read_status();
        if (stv) { g_layer_error = "a bounded device-side wait gave up (code " + std::to_string(stv) + ")"; return RESIST_ETIMEOUT; } }
    return RESIST_OK;
}
