// Launch plans of the local training step (Algorithm 1, inner loop) and of evaluation (Sec. 2.6).
// For a given partition and batch size every sub-ResNet is unrolled into a list of keyed operations;
// operations of different sub-ResNets with the same key become ONE grouped launch whose blockIdx.y
// selects the sub-ResNet, so that S shallow networks fill the GPU together.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include "runtime.h"

namespace resist {

void* ctx_alloc(resist_ctx* ctx, size_t bytes);
void ctx_free(resist_ctx* ctx, void* p);
void held_segments(const resist_ctx* ctx, int sub, uint32_t bit, bool buffers, std::vector<Segment>& out, long long& chunks);
int ensure_param_arrays(resist_ctx* ctx, int S);
int ensure_seg_table(resist_ctx* ctx, int n);
bool conv_tc_supported(const ConvProb& p, int mode);                                   // conv_tc.cu
int conv_tc_fill(const ConvProb& p, int mode, void* host_tc);
int conv_tc_count(const ConvProb& p, int mode);
int conv_tc_stat_tiles(const ConvProb& p);
int bn_fused_capacity(int backward);                                                    // kernels_ref.cu
void launch_bn_finalize_tiles(const BnProb* d, int nprob, int max_c, cudaStream_t s);
size_t conv_tc_prob_bytes();
int conv_tc_tiles(const void* host_tc);
size_t conv_tc_smem(const void* host_tc);
size_t conv_tc_merge(size_t a, size_t b);
void launch_conv_tc_probs(const void* d_tc, int nprob, int max_tiles, size_t max_smem, cudaStream_t s);
bool conv_wgrad_tc_supported(const ConvProb& p, int target_ctas, size_t* partial_bytes);
bool conv_wgrad_tc_fill(const ConvProb& p, int target_ctas, void* host_tc);
size_t conv_wgrad_tc_prob_bytes();
int conv_wgrad_tc_ctas(const void* h);
size_t conv_wgrad_tc_smem(const void* h);
long long conv_wgrad_tc_out_elems(const void* h);
void launch_conv_wgrad_tc_probs(const void* d_tc, int nprob, int max_ctas, size_t max_smem, long long max_out, cudaStream_t s);
// CTAs per weight-gradient problem so that a launch of nprob problems fills the GPU; the partial-sum workspace is sized for
// a problem launched alone (nprob = 1, the default)
static int wgrad_target_ctas(const resist_ctx* ctx, int nprob = 1) { return std::max(8, 2 * ctx->sm_count / std::max(1, nprob)); }
bool conv_mma_supported(const ConvProb& p, int mode);                                   // conv_mma.cu
bool conv_mma_fill(const ConvProb& p, int mode, void* host, const BnProb* bn = nullptr);
bool conv_mma_can_fuse_bn(const ConvProb& p, int mode, int C);
size_t conv_mma_bn_partial_bytes(int C, int sms);
size_t conv_mma_prob_bytes();
int conv_mma_tiles(const void* h);
size_t conv_mma_smem(const void* h);
bool launch_conv_mma_probs(const void* d, int nprob, int max_tiles, size_t max_smem, int variant, cudaStream_t s, bool pdl = false);
constexpr int MMA_BACKEND_FUSED = 512;                       // added to a warp-MMA forward/dgrad backend value: the consuming BN runs in the same launch
int conv_mma_pick_variant(const ConvProb& p, int mode);
bool conv_wgrad_mma_supported(const ConvProb& p, int target_ctas, size_t* partial_bytes);
bool conv_wgrad_mma_fill(const ConvProb& p, int target_ctas, void* host);
size_t conv_wgrad_mma_prob_bytes();
int conv_wgrad_mma_ctas(const void* h);
size_t conv_wgrad_mma_smem(const void* h);
long long conv_wgrad_mma_out_elems(const void* h);
void launch_conv_wgrad_mma_probs(const void* d, int nprob, int max_ctas, size_t max_smem, long long max_out, int variant, cudaStream_t s, bool pdl = false);
int conv_wgrad_mma_pick_variant(const ConvProb& p, int target_ctas);

// Which kernel family takes a bf16 convolution: 0 = CUDA cores, 1 = tcgen05, >= 200 = warp-level MMA (wgrad: 200 +
// output channels; forward and dgrad: 1000 + the kernel variant, so that the value also separates launches by what
// the kernel is specialised on).
static int pick_backend(const ConvProb& p, int mode, int target_ctas, size_t* partial_bytes, int pref = RESIST_CONV_AUTO) {
    bool want_mma = pref == RESIST_CONV_AUTO || pref == RESIST_CONV_WARP_MMA || pref == RESIST_CONV_WARP_MMA_UNFUSED; const bool want_tc = pref == RESIST_CONV_AUTO || pref == RESIST_CONV_TCGEN05;
    // 3x3 layers of 64 channels and more with many positions run faster on tcgen05 followed by the streaming BN kernels than on
    // the warp-level MMA kernels with the BN inside (measured at 8 x 128 images of 32 x 32: 450 -> 218 us forward, 668 -> 211 +
    // 195 us backward); small ones stay (a ResNet-110 stage of 8 x 8 maps measured the same either way)
    if (pref == RESIST_CONV_AUTO && p.C >= 64 && p.K >= 64 && p.ksz == 3 && (long long)p.N * p.H * p.W >= 65536) want_mma = false;
    if (mode == CONV_WGRAD) {
        if (want_mma && conv_wgrad_mma_supported(p, target_ctas, partial_bytes)) return 200 + conv_wgrad_mma_pick_variant(p, target_ctas);
        if (want_tc && conv_wgrad_tc_supported(p, target_ctas, partial_bytes)) return 1;
        return 0;
    }
    if (want_mma && conv_mma_supported(p, mode)) return 1000 + conv_mma_pick_variant(p, mode);
    if (want_tc && conv_tc_supported(p, mode)) return 1;
    return 0;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static int out_dim(int h, int k, int stride) { return (h + 2 * ((k - 1) / 2) - k) / stride + 1; }

void free_plan(resist_ctx* ctx, Plan& p) {
    ctx_free(ctx, p.d_blob);
    p = Plan();
}

struct PatchArgs {
    const void* images[RESIST_MAX_SUBNETS]; const int* labels[RESIST_MAX_SUBNETS];
    float* loss_out; float* logits_out; int* correct;
};
__global__ void patch_kernel(const PatchSite* sites, int n, PatchArgs a) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const PatchSite s = sites[i];
    void* v = nullptr;
    if (s.what == 0) v = (void*)a.images[s.sub];
    else if (s.what == 1) v = (void*)a.labels[s.sub];
    else if (s.what == 2) v = a.loss_out ? (void*)(a.loss_out + s.sub) : nullptr;
    else if (s.what == 3) v = (void*)a.logits_out;
    else v = (void*)a.correct;
    *s.where = v;
}

// ------------------------------------------------------------------------------------------------
// Unrolling one sub-ResNet into operations.  Device memory comes from a bump allocator over the
// sub-ResNet's workspace slice; with base == nullptr the pass only measures.
// ------------------------------------------------------------------------------------------------
struct Builder {
    resist_ctx* ctx; int B; int sub; int copy; bool eval; int slot_for_patch;
    char* base; size_t off = 0; size_t es;
    std::vector<Op>* ops;
    // scratch shared by the operations of this sub-ResNet (they run one after another)
    double* bn_partial = nullptr; float* wgrad_partial = nullptr; size_t bn_partial_need = 0, wgrad_partial_need = 0;
    char* up_buf = nullptr; size_t up_need = 0; const void* up_src = nullptr;      // zero-stuffed dy of the current stride-2 layer
    char* col_buf = nullptr; char* col_w = nullptr;                                 // im2col of the input images and the stem's weights packed alike
    static constexpr int NGBUF = 12;           // rotating gradient buffers: the more, the further the main stream runs ahead of the weight gradients
    char* gbuf[NGBUF] = {}; bool gused[NGBUF] = {}; size_t gbig = 0;
    float* logits = nullptr;
    long long flops = 0; int n_tc = 0, n_cc = 0;
    // The BN+ReLU that consumes a warp-MMA convolution's output joins that convolution's launch (forward: the BN of the
    // output; backward: the BN backward whose da the data gradient produces).  Index of the candidate in *ops, or -1.
    int last_fwd_conv = -1, last_dgrad = -1;
    int last_tc_fwd = -1;     // the last forward convolution if it runs on tcgen05: its epilogue can leave the sums the BN of its output needs
    bool fusable(int idx, const void* tensor, const BnProb& p) const {
        if (idx < 0 || eval || ctx->opts.dtype != RESIST_BF16 || (ctx->opts.conv_backend != RESIST_CONV_AUTO && ctx->opts.conv_backend != RESIST_CONV_WARP_MMA)) return false;
        const Op& o = (*ops)[idx];
        const int cout = o.kind == OP_CONV_FWD ? o.conv.K : o.conv.C;
        return o.backend >= 1000 && o.conv.out == tensor && p.vec && p.C == cout && conv_mma_can_fuse_bn(o.conv, o.kind == OP_CONV_FWD ? CONV_FWD : CONV_DGRAD, p.C);
    }

    void* take(size_t bytes) { off = align_up(off, 256); void* p = base ? base + off : nullptr; off += bytes; return p; }
    void* act(long long elems) { size_t b = (size_t)elems * es; if (b > gbig) gbig = b; return take(b); }
    // gradient buffers are handed out oldest-released first: a weight gradient that still reads a released buffer on
    // the second stream then has several layers' time before the buffer is written again
    int gstamp[NGBUF] = {}; int gclock = 0;
    int gtake() { int best = -1; for (int i = 0; i < NGBUF; ++i) if (!gused[i] && (best < 0 || gstamp[i] < gstamp[best])) best = i; if (best >= 0) gused[best] = true; return best; }
    void grel(int i) { if (i >= 0) { gused[i] = false; gstamp[i] = ++gclock; } }

    float* W() const { return ctx->pa.w + (long long)copy * ctx->pa.n; }
    float* G() const { return ctx->pa.g + (long long)copy * ctx->pa.n; }
    float* Bf() const { return ctx->pa.buf + (long long)copy * ctx->pa.nbuf; }
    const void* CW(long long o) const {           // the convolutions' copy of the weights
        if (ctx->opts.dtype == RESIST_BF16) return ctx->pa.wb + (long long)copy * ctx->pa.n + o;
        return W() + o;
    }

    // add_compact: `add` holds the gradient at the even positions only ([N,(H+1)/2,(W+1)/2,C], what a stride-2 projection's dgrad on
    // tcgen05 leaves).  Returns whether THIS convolution's output is such a compact tensor.
    bool conv(long long key, int mode, const void* a, const ConvRef& cr, const void* dy_or_null, const void* add, void* out,
              int N, int H, int Wd, float scale, bool patch = false, bool add_compact = false) {
        Op op{}; op.key = key; op.sub = sub; op.patch_images = patch ? 1 : 0;
        op.kind = mode == CONV_FWD ? OP_CONV_FWD : mode == CONV_DGRAD ? OP_CONV_DGRAD : OP_CONV_WGRAD;
        ConvProb& p = op.conv;
        p.N = N; p.H = H; p.W = Wd; p.C = cr.cin; p.K = cr.cout; p.ksz = cr.k; p.stride = cr.stride; p.pad = (cr.k - 1) / 2;
        p.P = out_dim(H, cr.k, cr.stride); p.Q = out_dim(Wd, cr.k, cr.stride);
        p.scale = scale; p.add = add; p.out = out; p.partial = nullptr;
        const long long rows_out = (long long)N * p.P * p.Q, rows_in = (long long)N * H * Wd;
        if (mode == CONV_FWD) { p.act = a; p.wgt = CW(cr.w); p.M = (int)rows_out; p.Ncol = p.K; p.Kred = p.ksz * p.ksz * p.C; }
        else if (mode == CONV_DGRAD) { p.act = dy_or_null; p.wgt = CW(cr.w); p.M = (int)rows_in; p.Ncol = p.C; p.Kred = p.ksz * p.ksz * p.K; }
        else { p.act = a; p.wgt = dy_or_null; p.M = p.K; p.Ncol = p.ksz * p.ksz * p.C; p.Kred = (int)rows_out; p.out = G() + cr.w; }
        p.tiles_m = (p.M + 63) / 64; p.tiles_n = (p.Ncol + 63) / 64; p.splits = 1;
        const int ktiles = (p.Kred + 15) / 16; p.ktiles_per_split = ktiles;
        flops += 2LL * rows_out * p.K * p.ksz * p.ksz * p.C;
        const bool tc_ok = ctx->opts.dtype == RESIST_BF16 && ctx->opts.conv_backend != RESIST_CONV_CUDA_CORES;
        const int pref = ctx->opts.conv_backend;
        if (tc_ok && p.stride == 2 && mode != CONV_FWD && !patch && p.K % 8 == 0) {
            // backward of a stride-2 layer on the warp-MMA kernels: a stride-1 problem that reads the compact dy through its pixel
            // tables (odd positions are zero); the tcgen05 kernels take the stride-2 problem as it is
            ConvProb q = p; q.stride = 1; q.P = p.H; q.Q = p.W; q.dy_sub = 2; q.dy_P = p.P; q.dy_Q = p.Q;
            if (mode == CONV_DGRAD) q.M = (int)rows_in; else q.Kred = (int)rows_in;
            size_t pb = 0;
            if (pick_backend(q, mode, wgrad_target_ctas(ctx), &pb, pref) >= 200) {
                p = q;
                if (mode == CONV_WGRAD) wgrad_partial_need = std::max(wgrad_partial_need, pb);
            }
        }
        if (mode == CONV_WGRAD) {
            size_t pb = 0;
            op.backend = (tc_ok && !patch) ? pick_backend(p, mode, wgrad_target_ctas(ctx), &pb, pref) : 0;
            if (op.backend) { wgrad_partial_need = std::max(wgrad_partial_need, pb); p.partial = wgrad_partial; }
        } else op.backend = tc_ok ? pick_backend(p, mode, 0, nullptr, pref) : 0;
        if (op.backend) ++n_tc; else ++n_cc;
        const bool out_compact = mode == CONV_DGRAD && op.backend == 1 && p.ksz == 1 && p.stride == 2;
        if (out_compact) p.out_compact = 1;
        if (add && add_compact) {
            if (op.backend == 1 && mode == CONV_DGRAD) p.add_sub = 2;            // added at the even positions in the epilogue
            else {                                                               // spread out to the full resolution first
                up_need = std::max(up_need, (size_t)rows_in * p.C * 2);
                Op u{}; u.key = key; u.sub = sub; u.kind = OP_UPSAMPLE;
                u.up = UpProb{add, up_buf, N, H, Wd, p.C, (H + 1) / 2, (Wd + 1) / 2};
                ops->push_back(u); p.add = up_buf;
            }
        }
        if (mode == CONV_WGRAD && !op.backend) {
            const int tiles = p.tiles_m * p.tiles_n;
            int want = (2 * ctx->sm_count + tiles - 1) / tiles; if (want > 64) want = 64; if (want > ktiles) want = ktiles; if (want < 1) want = 1;
            p.ktiles_per_split = (ktiles + want - 1) / want; p.splits = (ktiles + p.ktiles_per_split - 1) / p.ktiles_per_split;
            if (p.splits > 1) {
                wgrad_partial_need = std::max(wgrad_partial_need, (size_t)p.splits * p.M * p.Ncol * 4);
                p.partial = wgrad_partial;
            }
        }
        ops->push_back(op);
        if (mode == CONV_FWD) { last_fwd_conv = op.backend >= 1000 ? (int)ops->size() - 1 : -1; last_tc_fwd = op.backend == 1 ? (int)ops->size() - 1 : -1; }
        if (mode == CONV_DGRAD) last_dgrad = op.backend >= 1000 ? (int)ops->size() - 1 : -1;
        if (mode == CONV_WGRAD && p.splits > 1) { Op r = op; r.key = key + 1; r.kind = OP_SPLITK; r.patch_images = 0; ops->push_back(r); }
        return out_compact;
    }
    // the BN joins the launch of the convolution at *ops[idx]
    void fuse_into(int idx, const BnProb& p, int which) {
        Op& o = (*ops)[idx];
        o.fuse = which; o.bn = p; o.backend += MMA_BACKEND_FUSED;
        bn_partial_need = std::max(bn_partial_need, conv_mma_bn_partial_bytes(p.C, ctx->sm_count));
        o.bn.partial = bn_partial;
    }

    // A stem with few input channels (bf16): the images are expanded once per step to rows of (tap, channel) columns, and forward
    // and wgrad become 1x1 problems on the tensor-core kernels.  Up to 32 columns (3x3 stems of 3 channels): rows of 32 on the
    // warp-MMA kernels.  More (7x7 stems: 147 columns, pitch 152): on the tcgen05 kernels, whose TMA fills the last 64-column
    // slab with zeros; the weight gradient is computed at the row pitch and repacked.
    int stem_cols(const ConvRef& cr) const {
        if (ctx->opts.dtype != RESIST_BF16 || ctx->opts.conv_backend == RESIST_CONV_CUDA_CORES) return 0;
        const int kk = cr.cin * cr.k * cr.k, pref = ctx->opts.conv_backend;
        if (kk <= 32 && cr.cout % 16 == 0 && cr.cout <= 64 && pref != RESIST_CONV_TCGEN05) return 32;
        if (kk > 32 && kk <= 256 && cr.cin < 8 && cr.cout % 8 == 0 && (pref == RESIST_CONV_AUTO || pref == RESIST_CONV_TCGEN05)) return (kk + 7) / 8 * 8;
        return 0;
    }
    bool stem_as_im2col(const ConvRef& cr) const { return stem_cols(cr) != 0; }
    float* stem_dw = nullptr;                                     // wide stem: weight gradient at the row pitch, before repacking
    void stem_im2col(long long key, const ConvRef& cr, int N, int H, int Wd) {
        const int P = out_dim(H, cr.k, cr.stride), Q = out_dim(Wd, cr.k, cr.stride), cols = stem_cols(cr);
        col_buf = (char*)take((size_t)N * P * Q * cols * 2); col_w = (char*)take((size_t)cr.cout * cols * 2);
        if (cols > 32) stem_dw = (float*)take((size_t)cr.cout * cols * 4);
        Op u{}; u.key = key; u.sub = sub; u.kind = OP_IM2COL;
        u.col = ColProb{nullptr, col_buf, CW(cr.w), col_w, N, H, Wd, cr.cin, cr.k, cr.stride, (cr.k - 1) / 2, P, Q, cr.cout, cr.cin * cr.k * cr.k, cols};
        ops->push_back(u);
    }
    // the stem as a 1x1 problem on the im2col'ed images: forward (out = y) or wgrad (dy given; dw goes to the stem's gradient)
    void stem_conv(long long key, int mode, const ConvRef& cr, const void* dy, void* out, int N, int H, int Wd) {
        const int P = out_dim(H, cr.k, cr.stride), Q = out_dim(Wd, cr.k, cr.stride), cols = stem_cols(cr), kk = cr.cin * cr.k * cr.k;
        const bool wide = cols > 32;
        Op op{}; op.key = key; op.sub = sub; op.kind = mode == CONV_FWD ? OP_CONV_FWD : OP_CONV_WGRAD;
        ConvProb& p = op.conv;
        p.N = N; p.H = P; p.W = Q; p.C = cols; p.K = cr.cout; p.ksz = 1; p.stride = 1; p.pad = 0; p.P = P; p.Q = Q; p.scale = 1.f;
        const long long rows = (long long)N * P * Q;
        p.act = col_buf;
        if (mode == CONV_FWD) { p.wgt = col_w; p.out = out; p.M = (int)rows; p.Ncol = p.K; p.Kred = cols; }
        else { p.wgt = dy; p.out = wide ? stem_dw : G() + cr.w; p.M = p.K; p.Ncol = cols; p.Kred = (int)rows; if (!wide) { p.wg_ld = kk; p.wg_cols = kk; } }
        p.tiles_m = (p.M + 63) / 64; p.tiles_n = (p.Ncol + 63) / 64; p.splits = 1; p.ktiles_per_split = (p.Kred + 15) / 16;
        flops += 2LL * rows * p.K * kk;
        size_t pb = 0;
        op.backend = pick_backend(p, mode, wgrad_target_ctas(ctx), &pb, wide ? RESIST_CONV_TCGEN05 : RESIST_CONV_WARP_MMA);
        if (mode == CONV_WGRAD) { wgrad_partial_need = std::max(wgrad_partial_need, pb); p.partial = wgrad_partial; }
        ++n_tc;
        ops->push_back(op);
        if (mode == CONV_FWD) { last_fwd_conv = op.backend >= 1000 ? (int)ops->size() - 1 : -1; last_tc_fwd = op.backend == 1 ? (int)ops->size() - 1 : -1; }
        if (mode == CONV_WGRAD && wide) {                      // [K][cols] -> the stem's [K][k][k][C] in the gradient vector
            Op r{}; r.key = key + 1; r.sub = sub; r.kind = OP_REPACK;
            r.conv.act = stem_dw; r.conv.out = G() + cr.w; r.conv.M = cr.cout; r.conv.Ncol = kk; r.conv.Kred = cols;
            ops->push_back(r);
        }
    }

    // chunks per BN problem that give the fused (cooperative) kernels about two CTAs per SM over all sub-ResNets
    int fused_chunks() const { return std::max(8, 2 * ctx->sm_count / std::max(1, ctx->S)); }
    // forward BN+ReLU: statistics (or running statistics in evaluation) then apply
    float* bn_fwd(long long key, const void* x, void* a, const BNRef& r, long long m) {
        float* stat = (float*)take((size_t)4 * r.c * 4);
        Op op{}; op.key = key; op.sub = sub; op.kind = OP_BN_STATS;
        BnProb& p = op.bn;
        p.x = x; p.a = a; p.gamma = W() + r.g; p.beta = W() + r.b; p.dgamma = G() + r.g; p.dbeta = G() + r.b;
        p.run_mean = Bf() + r.buf; p.run_var = Bf() + r.buf + r.c; p.stat = stat; p.m = m; p.C = r.c;
        p.eps = ctx->opts.bn_eps; p.momentum = ctx->opts.bn_momentum; p.eval = eval ? 1 : 0;
        bn_chunking(p, ctx->opts.dtype == RESIST_BF16, fused_chunks());
        bn_partial_need = std::max(bn_partial_need, (size_t)p.chunks * 2 * r.c * 8);
        p.partial = bn_partial;
        const int producer = last_fwd_conv; last_fwd_conv = -1;
        const int tc_producer = last_tc_fwd; last_tc_fwd = -1;
        if (fusable(producer, x, p)) { fuse_into(producer, p, 1); return stat; }                            // inside the producing convolution's launch
        if (!eval && p.vec && tc_producer >= 0 && (*ops)[tc_producer].conv.out == x && (*ops)[tc_producer].conv.K == r.c) {
            // the tcgen05 convolution that produces x leaves per-tile column sums: a small launch turns them into statistics, then one elementwise pass
            ConvProb& c = (*ops)[tc_producer].conv;
            const int tiles = conv_tc_stat_tiles(c);
            bn_partial_need = std::max(bn_partial_need, (size_t)tiles * 2 * r.c * 4);
            c.stat_tiles = (float*)bn_partial; p.partial = bn_partial; p.chunks = tiles;
            op.kind = OP_BN_TILE_STATS; ops->push_back(op);
            op.key = key + 1; op.kind = OP_BN_APPLY; ops->push_back(op);
            return stat;
        }
        if (p.vec && !eval && r.c <= 512 && (long long)p.chunks * ctx->S <= bn_fused_capacity(0)) { op.kind = OP_BN_FWD_FUSED; ops->push_back(op); return stat; }   // one cooperative launch
        ops->push_back(op);
        op.key = key + 1; op.kind = OP_BN_APPLY; ops->push_back(op);
        return stat;
    }
    void bn_bwd(long long key, const void* x, const void* da, void* dx, const void* add, const BNRef& r, float* stat, long long m) {
        Op op{}; op.key = key; op.sub = sub; op.kind = OP_BN_BWD_REDUCE;
        BnProb& p = op.bn;
        p.x = x; p.da = da; p.dx = dx; p.add = add; p.gamma = W() + r.g; p.beta = W() + r.b; p.dgamma = G() + r.g; p.dbeta = G() + r.b;
        p.stat = stat; p.m = m; p.C = r.c; p.eps = ctx->opts.bn_eps; p.momentum = ctx->opts.bn_momentum; p.eval = 0;
        // (measured on 8 x 67 MB tensors, far beyond L2: reduction + elementwise pass as two streaming launches, each with twelve
        // 16-byte loads in flight per thread and two CTAs per SM, take 194 + 323 us; the cooperative kernel with three CTAs per SM and one
        // row in flight took 794 us; both move the same five passes over HBM, so the cooperative form only pays for tensors that
        // stay in L2 between its two passes)
        bn_chunking(p, ctx->opts.dtype == RESIST_BF16, fused_chunks());
        bn_partial_need = std::max(bn_partial_need, (size_t)p.chunks * 2 * r.c * 8);
        p.partial = bn_partial;
        const int producer = last_dgrad; last_dgrad = -1;
        if (fusable(producer, da, p)) { fuse_into(producer, p, 2); return; }
        // one cooperative launch where all sub-ResNets' chunks can be resident together (the kernel holds 128 registers: one CTA
        // per SM), else the reduction and the elementwise pass as launches of their own
        if (p.vec && r.c <= 512 && (long long)p.chunks * ctx->S <= bn_fused_capacity(1)) { op.kind = OP_BN_BWD_FUSED; ops->push_back(op); return; }
        if (p.vec) {
            // the reduction as a launch of its own: about four waves of CTAs over all sub-ResNets (long enough chunks for the batched
            // loads to pipeline, enough of them for the SMs to even out the tail)
            const int R = 256 / (r.c / 8);
            long long rpc = (m + 4 * fused_chunks() - 1) / (4 * fused_chunks());
            rpc = (rpc + R - 1) / R * R; if (rpc < 32 * R) rpc = 32 * R;
            if (rpc > p.rows_per_chunk) { p.rows_per_chunk = (int)rpc; p.chunks = (int)((m + rpc - 1) / rpc); }
        }
        ops->push_back(op);
        op.key = key + 1; op.kind = OP_BN_BWD_APPLY; ops->push_back(op);
    }
};

struct BlockMem { int H, W, Ho, Wo; void *x, *a1, *y1, *a2, *y2, *a3; float* stat[3]; };

// Returns the workspace bytes this sub-ResNet needs.  `present` has one entry per block.
static size_t unroll_subnet(resist_ctx* ctx, Builder& bd, const std::vector<char>& present, float inv_S) {
    const resist_arch& A = ctx->arch; const Layout& L = ctx->L; const int B = bd.B; const int nb = A.num_blocks;
    const long long KEY_BLOCK0 = 100, FWD_END = KEY_BLOCK0 + 20LL * nb, BWD0 = FWD_END + 10, BWD_BLOCK0 = BWD0 + 10;
    const long long BWD_END = BWD_BLOCK0 + 40LL * nb;
    // scratch first, so that its addresses do not depend on the network above it
    bd.bn_partial = (double*)bd.take(bd.bn_partial_need);
    bd.wgrad_partial = (float*)bd.take(bd.wgrad_partial_need);
    bd.up_buf = (char*)bd.take(bd.up_need);
    if (!bd.eval) for (int i = 0; i < Builder::NGBUF; ++i) bd.gbuf[i] = (char*)bd.take(bd.gbig);

    // ---- stem
    const int Hs = out_dim(A.in_h, A.stem_k, A.stem_stride), Ws = out_dim(A.in_w, A.stem_k, A.stem_stride);
    const long long m_stem = (long long)B * Hs * Ws;
    void* stem_y = bd.act(m_stem * A.stem_cout); void* stem_a = nullptr; void* stem_p = nullptr; int* stem_arg = nullptr; float* stem_stat = nullptr;
    const bool stem_col = bd.stem_as_im2col(L.stem);
    if (stem_col) { bd.stem_im2col(0, L.stem, B, A.in_h, A.in_w); bd.stem_conv(0, CONV_FWD, L.stem, nullptr, stem_y, B, A.in_h, A.in_w); }
    else bd.conv(0, CONV_FWD, nullptr, L.stem, nullptr, nullptr, stem_y, B, A.in_h, A.in_w, 1.f, true);
    void* cur = stem_y; int cH = Hs, cW = Ws, cC = A.stem_cout;
    if (A.stem_bn_relu) { stem_a = bd.act(m_stem * cC); stem_stat = bd.bn_fwd(1, stem_y, stem_a, L.stem_bn, m_stem); cur = stem_a; }
    if (A.stem_maxpool) {
        const int Hp = out_dim(cH, 3, 2), Wp = out_dim(cW, 3, 2);
        stem_p = bd.act((long long)B * Hp * Wp * cC); stem_arg = (int*)bd.take((size_t)B * Hp * Wp * cC * 4);
        Op op{}; op.key = 3; op.sub = bd.sub; op.kind = OP_POOL_FWD;
        op.pool = PoolProb{cur, stem_p, stem_arg, nullptr, nullptr, B, cH, cW, cC, Hp, Wp};
        bd.ops->push_back(op); bd.last_fwd_conv = -1; bd.last_tc_fwd = -1;
        cur = stem_p; cH = Hp; cW = Wp;
    }

    // ---- blocks
    std::vector<BlockMem> bm(nb); std::vector<int> order;
    for (int b = 0; b < nb; ++b) if (present[b]) order.push_back(b);
    // Launch slots are aligned by stage: the i-th present block of stage t gets slot base(t) + i, where base(t) adds up, over
    // the earlier stages, the largest number of blocks any sub-ResNet of this round holds there.  Sub-ResNets then share a
    // launch only with blocks of the same stage (same shapes, same kernel variant), instead of splitting a slot's launch
    // whenever their block counts per stage differ.
    std::vector<int> aslot(order.size(), 0); int n_aslots = 0;
    {
        int n_stage = 0; for (int b = 0; b < nb; ++b) n_stage = std::max(n_stage, ctx->blocks[b].stage + 1);
        std::vector<int> stage_max(std::max(n_stage, 1), 0), cnt(std::max(n_stage, 1), 0);
        for (int b = 0; b < nb; ++b) if (present[b]) ++cnt[std::max(0, ctx->blocks[b].stage)];
        stage_max = cnt;
        for (int s2 = 0; s2 < ctx->S && (int)ctx->mask.size() == nb; ++s2) {
            std::fill(cnt.begin(), cnt.end(), 0);
            for (int b = 0; b < nb; ++b) if (ctx->mask[b] >> s2 & 1u) ++cnt[std::max(0, ctx->blocks[b].stage)];
            for (size_t t = 0; t < cnt.size(); ++t) stage_max[t] = std::max(stage_max[t], cnt[t]);
        }
        std::vector<int> base(stage_max.size() + 1, 0);
        for (size_t t = 0; t < stage_max.size(); ++t) base[t + 1] = base[t] + stage_max[t];
        n_aslots = base.back();
        std::fill(cnt.begin(), cnt.end(), 0);
        for (size_t i = 0; i < order.size(); ++i) { const int t = std::max(0, ctx->blocks[order[i]].stage); aslot[i] = base[t] + cnt[t]++; }
    }
    for (size_t slot = 0; slot < order.size(); ++slot) {
        const int b = order[slot]; const resist_block& K = ctx->blocks[b]; const BlockRef& r = L.blk[b]; BlockMem& s = bm[b];
        const long long key = KEY_BLOCK0 + 20LL * (long long)aslot[slot];
        s.H = cH; s.W = cW; s.Ho = out_dim(cH, 3, K.stride); s.Wo = out_dim(cW, 3, K.stride);
        const long long m_in = (long long)B * s.H * s.W, m_out = (long long)B * s.Ho * s.Wo;
        const float scale = (bd.eval && K.partitionable) ? inv_S : 1.f;
        s.x = cur; s.a1 = bd.act(m_in * K.cin);
        s.stat[0] = bd.bn_fwd(key + 0, s.x, s.a1, r.bn[0], m_in);
        const void* sc = s.x;
        if (K.has_projection) { void* scb = bd.act(m_out * K.cout); bd.conv(key + 2, CONV_FWD, s.a1, r.proj, nullptr, nullptr, scb, B, s.H, s.W, 1.f); sc = scb; }
        void* out = bd.act(m_out * K.cout);
        if (K.kind == RESIST_BASIC) {
            s.y1 = bd.act(m_out * K.cout); s.a2 = bd.act(m_out * K.cout);
            bd.conv(key + 3, CONV_FWD, s.a1, r.conv[0], nullptr, nullptr, s.y1, B, s.H, s.W, 1.f);
            s.stat[1] = bd.bn_fwd(key + 4, s.y1, s.a2, r.bn[1], m_out);
            bd.conv(key + 6, CONV_FWD, s.a2, r.conv[1], nullptr, sc, out, B, s.Ho, s.Wo, scale);
        } else {
            s.y1 = bd.act(m_in * K.cmid); s.a2 = bd.act(m_in * K.cmid); s.y2 = bd.act(m_out * K.cmid); s.a3 = bd.act(m_out * K.cmid);
            bd.conv(key + 3, CONV_FWD, s.a1, r.conv[0], nullptr, nullptr, s.y1, B, s.H, s.W, 1.f);
            s.stat[1] = bd.bn_fwd(key + 4, s.y1, s.a2, r.bn[1], m_in);
            bd.conv(key + 6, CONV_FWD, s.a2, r.conv[1], nullptr, nullptr, s.y2, B, s.H, s.W, 1.f);
            s.stat[2] = bd.bn_fwd(key + 7, s.y2, s.a3, r.bn[2], m_out);
            bd.conv(key + 9, CONV_FWD, s.a3, r.conv[2], nullptr, sc, out, B, s.Ho, s.Wo, scale);
        }
        cur = out; cH = s.Ho; cW = s.Wo; cC = K.cout;
    }

    // ---- final BN + ReLU, pool, head, loss
    const long long mF = (long long)B * cH * cW; const int HW = cH * cW;
    void* xF = cur; void* aF = bd.act(mF * cC);
    float* statF = bd.bn_fwd(FWD_END, xF, aF, L.final_bn, mF);
    HeadProb hp{};
    hp.a = aF; hp.w = bd.W() + L.head_w; hp.b = bd.W() + L.head_b; hp.dw = bd.G() + L.head_w; hp.db = bd.G() + L.head_b;
    hp.pooled = (float*)bd.take((size_t)B * cC * 4); hp.dpooled = (float*)bd.take((size_t)B * cC * 4);
    hp.logits = (float*)bd.take((size_t)B * A.classes * 4); hp.dlogits = bd.eval ? nullptr : (float*)bd.take((size_t)B * A.classes * 4);
    hp.loss = (float*)bd.take(256); hp.B = B; hp.HW = HW; hp.C = cC; hp.classes = A.classes;
    bd.logits = hp.logits;
    { Op op{}; op.key = FWD_END + 2; op.sub = bd.sub; op.kind = OP_HEAD_FWD; op.head = hp; bd.ops->push_back(op); }
    if (bd.eval) return bd.off;

    // ---- backward
    int g_cur = bd.gtake();                                   // gradient w.r.t. the current tensor
    hp.da = bd.gbuf[g_cur];
    { Op op{}; op.key = BWD0; op.sub = bd.sub; op.kind = OP_HEAD_BWD; op.head = hp; bd.ops->push_back(op); }
    { int g = bd.gtake(); bd.bn_bwd(BWD0 + 1, xF, bd.gbuf[g_cur], bd.gbuf[g], nullptr, L.final_bn, statF, mF); bd.grel(g_cur); g_cur = g; }
    for (int slot = (int)order.size() - 1; slot >= 0; --slot) {
        const int b = order[slot]; const resist_block& K = ctx->blocks[b]; const BlockRef& r = L.blk[b]; BlockMem& s = bm[b];
        const long long key = BWD_BLOCK0 + 40LL * ((long long)n_aslots - 1 - aslot[slot]);
        const long long m_in = (long long)B * s.H * s.W, m_out = (long long)B * s.Ho * s.Wo;
        const char* dout = bd.gbuf[g_cur];
        bd.up_src = nullptr;                                     // no zero-stuffed dy carries over from another block
        int g_sc = -1; bool sc_compact = false;
        if (K.has_projection) {
            bd.conv(key + 0, CONV_WGRAD, s.a1, r.proj, dout, nullptr, nullptr, B, s.H, s.W, 1.f);
            g_sc = bd.gtake();
            sc_compact = bd.conv(key + 2, CONV_DGRAD, nullptr, r.proj, dout, nullptr, bd.gbuf[g_sc], B, s.H, s.W, 1.f);
        }
        int g_da1 = -1;
        if (K.kind == RESIST_BASIC) {
            const int g_da2 = bd.gtake();
            bd.conv(key + 3, CONV_WGRAD, s.a2, r.conv[1], dout, nullptr, nullptr, B, s.Ho, s.Wo, 1.f);
            bd.conv(key + 5, CONV_DGRAD, nullptr, r.conv[1], dout, nullptr, bd.gbuf[g_da2], B, s.Ho, s.Wo, 1.f);
            const int g_dy1 = bd.gtake();
            bd.bn_bwd(key + 6, s.y1, bd.gbuf[g_da2], bd.gbuf[g_dy1], nullptr, r.bn[1], s.stat[1], m_out);
            bd.grel(g_da2);
            bd.conv(key + 8, CONV_WGRAD, s.a1, r.conv[0], bd.gbuf[g_dy1], nullptr, nullptr, B, s.H, s.W, 1.f);
            g_da1 = bd.gtake();
            bd.conv(key + 10, CONV_DGRAD, nullptr, r.conv[0], bd.gbuf[g_dy1], g_sc >= 0 ? bd.gbuf[g_sc] : nullptr, bd.gbuf[g_da1], B, s.H, s.W, 1.f, false, sc_compact);
            bd.grel(g_dy1);
        } else {
            const int g_da3 = bd.gtake();
            bd.conv(key + 3, CONV_WGRAD, s.a3, r.conv[2], dout, nullptr, nullptr, B, s.Ho, s.Wo, 1.f);
            bd.conv(key + 5, CONV_DGRAD, nullptr, r.conv[2], dout, nullptr, bd.gbuf[g_da3], B, s.Ho, s.Wo, 1.f);
            const int g_dy2 = bd.gtake();
            bd.bn_bwd(key + 6, s.y2, bd.gbuf[g_da3], bd.gbuf[g_dy2], nullptr, r.bn[2], s.stat[2], m_out);
            bd.grel(g_da3);
            bd.conv(key + 8, CONV_WGRAD, s.a2, r.conv[1], bd.gbuf[g_dy2], nullptr, nullptr, B, s.H, s.W, 1.f);
            const int g_da2 = bd.gtake();
            bd.conv(key + 10, CONV_DGRAD, nullptr, r.conv[1], bd.gbuf[g_dy2], nullptr, bd.gbuf[g_da2], B, s.H, s.W, 1.f);
            bd.grel(g_dy2);
            const int g_dy1 = bd.gtake();
            bd.bn_bwd(key + 11, s.y1, bd.gbuf[g_da2], bd.gbuf[g_dy1], nullptr, r.bn[1], s.stat[1], m_in);
            bd.grel(g_da2);
            bd.conv(key + 13, CONV_WGRAD, s.a1, r.conv[0], bd.gbuf[g_dy1], nullptr, nullptr, B, s.H, s.W, 1.f);
            g_da1 = bd.gtake();
            bd.conv(key + 15, CONV_DGRAD, nullptr, r.conv[0], bd.gbuf[g_dy1], g_sc >= 0 ? bd.gbuf[g_sc] : nullptr, bd.gbuf[g_da1], B, s.H, s.W, 1.f, false, sc_compact);
            bd.grel(g_dy1);
        }
        bd.grel(g_sc);
        const int g_dx = bd.gtake();
        // identity skip: the block's input also receives dout directly
        bd.bn_bwd(key + 20, s.x, bd.gbuf[g_da1], bd.gbuf[g_dx], K.has_projection ? nullptr : dout, r.bn[0], s.stat[0], m_in);
        bd.grel(g_da1); bd.grel(g_cur); g_cur = g_dx;
    }
    // ---- stem backward (no input gradient)
    if (A.stem_maxpool) {
        const int g = bd.gtake();
        Op op{}; op.key = BWD_END; op.sub = bd.sub; op.kind = OP_POOL_BWD;
        op.pool = PoolProb{stem_a ? stem_a : stem_y, nullptr, stem_arg, bd.gbuf[g_cur], bd.gbuf[g], B, Hs, Ws, A.stem_cout, cH, cW};
        op.pool.P = out_dim(Hs, 3, 2); op.pool.Q = out_dim(Ws, 3, 2);
        bd.ops->push_back(op); bd.grel(g_cur); g_cur = g; bd.last_dgrad = -1;
    }
    if (A.stem_bn_relu) { const int g = bd.gtake(); bd.bn_bwd(BWD_END + 1, stem_y, bd.gbuf[g_cur], bd.gbuf[g], nullptr, L.stem_bn, stem_stat, m_stem); bd.grel(g_cur); g_cur = g; }
    if (stem_col) bd.stem_conv(BWD_END + 3, CONV_WGRAD, L.stem, bd.gbuf[g_cur], nullptr, B, A.in_h, A.in_w);
    else bd.conv(BWD_END + 3, CONV_WGRAD, nullptr, L.stem, bd.gbuf[g_cur], nullptr, nullptr, B, A.in_h, A.in_w, 1.f, true);
    return bd.off;
}

// ------------------------------------------------------------------------------------------------
// Workspace: one slice per sub-ResNet, all slices the size of the largest.
// ------------------------------------------------------------------------------------------------
struct Needs { size_t bn_partial = 0, wgrad_partial = 0, gbig = 0, up = 0, total = 0; };

static Needs measure_subnet(resist_ctx* ctx, int sub, int copy, const std::vector<char>& present, int B, bool eval, float inv_S) {
    std::vector<Op> scratch;
    Builder b1{ctx, B, sub, copy, eval, 0, nullptr}; b1.es = ctx->opts.dtype == RESIST_BF16 ? 2 : 4; b1.ops = &scratch;
    unroll_subnet(ctx, b1, present, inv_S);
    Needs n; n.bn_partial = b1.bn_partial_need; n.wgrad_partial = b1.wgrad_partial_need; n.gbig = b1.gbig; n.up = b1.up_need;
    scratch.clear();
    Builder b2{ctx, B, sub, copy, eval, 0, nullptr}; b2.es = b1.es; b2.ops = &scratch;
    b2.bn_partial_need = n.bn_partial; b2.wgrad_partial_need = n.wgrad_partial; b2.gbig = n.gbig; b2.up_need = n.up;
    n.total = align_up(unroll_subnet(ctx, b2, present, inv_S), 256);
    return n;
}

static std::vector<char> present_of(const resist_ctx* ctx, int sub) {
    std::vector<char> p(ctx->arch.num_blocks);
    for (int b = 0; b < ctx->arch.num_blocks; ++b) p[b] = (ctx->mask[b] >> sub & 1u) ? 1 : 0;
    return p;
}

static int upload_plan(resist_ctx* ctx, Plan& plan, std::vector<Op>& ops, bool single, cudaStream_t st) {
    // equal keys of different sub-ResNets become neighbours; a zero-stuffing or im2col op shares the key of the first
    // convolution that reads its output and sorts in front of it
    std::stable_sort(ops.begin(), ops.end(), [](const Op& a, const Op& b) {
        if (a.key != b.key) return a.key < b.key;
        const bool pa = a.kind == OP_UPSAMPLE || a.kind == OP_IM2COL, pb = b.kind == OP_UPSAMPLE || b.kind == OP_IM2COL;
        if (pa != pb) return pa;
        return a.backend < b.backend; });
    const double es = ctx->opts.dtype == RESIST_BF16 ? 2.0 : 4.0;
    std::vector<ConvProb> conv; std::vector<BnProb> bn; std::vector<PoolProb> pool; std::vector<HeadProb> head; std::vector<UpProb> up; std::vector<ColProb> col;
    const size_t tcb = conv_tc_prob_bytes(); std::vector<char> tc; int n_tc = 0;
    const size_t wtcb = conv_wgrad_tc_prob_bytes(); std::vector<char> wtc; int n_wtc = 0;
    const size_t mmb = conv_mma_prob_bytes(); std::vector<char> mm; int n_mm = 0;
    const size_t wmmb = conv_wgrad_mma_prob_bytes(); std::vector<char> wmm; int n_wmm = 0;
    struct HostSite { int arr; int idx; int field; int what; int sub; };
    std::vector<HostSite> sites;
    plan.launches.clear();
    std::vector<const void*> inflight;                         // tensors read by the weight gradients not yet joined
    for (size_t i = 0; i < ops.size();) {
        size_t j = i;
        while (j < ops.size() && ops[j].key == ops[i].key && ops[j].kind == ops[i].kind && ops[j].backend == ops[i].backend) ++j;
        Launch L{}; L.kind = ops[i].kind; L.backend = ops[i].backend; L.count = (int)(j - i);
        if (ops[i].kind == OP_CONV_FWD || ops[i].kind == OP_CONV_DGRAD || ops[i].kind == OP_CONV_WGRAD) {
            const ConvProb& c = ops[i].conv;
            snprintf(L.label, sizeof(L.label), "%dx%d C%d K%d HW%d s%d%s x%d", c.ksz, c.ksz, c.C, c.K, c.H, c.stride, c.dy_sub == 2 ? "*" : "", L.count);
        } else if (ops[i].kind != OP_HEAD_FWD && ops[i].kind != OP_HEAD_BWD && ops[i].kind != OP_POOL_FWD && ops[i].kind != OP_POOL_BWD &&
                   ops[i].kind != OP_UPSAMPLE && ops[i].kind != OP_IM2COL && ops[i].kind != OP_SPLITK && ops[i].kind != OP_REPACK)
            snprintf(L.label, sizeof(L.label), "bn m%lld C%d x%d", ops[i].bn.m, ops[i].bn.C, L.count);
        for (size_t k = i; k < j; ++k) {
            const Op& o = ops[k]; const int slot = single ? 0 : o.sub;
            switch (o.kind) {
                case OP_REPACK: {
                    if (k == i) L.first = (int)conv.size();
                    conv.push_back(o.conv);
                    L.max_elems = std::max<long long>(L.max_elems, (long long)o.conv.M * o.conv.Ncol); L.bytes += 8.0 * o.conv.M * o.conv.Ncol;
                    break; }
                case OP_CONV_FWD: case OP_CONV_DGRAD: case OP_CONV_WGRAD: case OP_SPLITK: {
                    if (o.backend >= 200 && o.kind != OP_SPLITK) {   // warp-level MMA kernels: their own descriptor arrays
                        const ConvProb& p = o.conv;
                        // algorithmic work of the layer itself: a stride-2 layer's dy has dy_P x dy_Q positions, whatever resolution the kernel walks
                        const double in_e = (double)p.N * p.H * p.W * p.C, out_e = (double)p.N * (p.dy_sub == 2 ? (double)p.dy_P * p.dy_Q : (double)p.P * p.Q) * p.K, w_e = (double)p.K * p.ksz * p.ksz * p.C;
                        L.flops += 2.0 * out_e * p.ksz * p.ksz * p.C;
                        if (o.kind == OP_CONV_WGRAD) {
                            if (k == i) L.first = n_wmm;
                            wmm.resize((size_t)(n_wmm + 1) * wmmb); char* h = wmm.data() + (size_t)n_wmm * wmmb;
                            if (!conv_wgrad_mma_fill(o.conv, wgrad_target_ctas(ctx, (int)(j - i)), h)) { ctx->err = "wgrad descriptor failed"; return RESIST_EINVAL; }
                            L.gx = std::max(L.gx, conv_wgrad_mma_ctas(h));
                            L.max_elems = std::max<long long>(L.max_elems, (long long)conv_wgrad_mma_smem(h));
                            L.max_b = (int)std::max<long long>(L.max_b, conv_wgrad_mma_out_elems(h));
                            ++n_wmm; L.bytes += es * (in_e + out_e) + 4.0 * w_e;
                        } else {
                            if (k == i) L.first = n_mm;
                            mm.resize((size_t)(n_mm + 1) * mmb); char* h = mm.data() + (size_t)n_mm * mmb;
                            const int mode = o.kind == OP_CONV_FWD ? CONV_FWD : CONV_DGRAD;
                            if (!conv_mma_fill(o.conv, mode, h, o.fuse ? &o.bn : nullptr)) { ctx->err = "conv descriptor failed"; return RESIST_EINVAL; }
                            L.gx = std::max(L.gx, conv_mma_tiles(h));
                            L.max_elems = std::max<long long>(L.max_elems, (long long)conv_mma_smem(h));
                            ++n_mm; L.bytes += es * (in_e + out_e + w_e + (p.add ? (o.kind == OP_CONV_FWD ? out_e : in_e) : 0.0));
                            // fused BN: forward writes a (its read of the output just written is an L2 hit); backward reads x (+ the skip gradient) and writes dx
                            if (o.fuse == 1) L.bytes += es * out_e;
                            if (o.fuse == 2) L.bytes += es * in_e * (o.bn.add ? 3 : 2);
                        }
                        break;
                    }
                    if (o.backend && o.kind == OP_CONV_WGRAD) {  // tensor-core wgrad: its own descriptor array
                        if (k == i) L.first = n_wtc;
                        wtc.resize((size_t)(n_wtc + 1) * wtcb);
                        char* h = wtc.data() + (size_t)n_wtc * wtcb;
                        if (!conv_wgrad_tc_fill(o.conv, wgrad_target_ctas(ctx, (int)(j - i)), h)) { ctx->err = "tensor map encoding failed"; return RESIST_ECUDA; }
                        L.gx = std::max(L.gx, conv_wgrad_tc_ctas(h));
                        L.max_elems = std::max<long long>(L.max_elems, (long long)conv_wgrad_tc_smem(h));
                        L.max_b = (int)std::max<long long>(L.max_b, conv_wgrad_tc_out_elems(h));
                        ++n_wtc;
                        const ConvProb& p = o.conv;
                        const double in_e = (double)p.N * p.H * p.W * p.C, out_e = (double)p.N * p.P * p.Q * p.K, w_e = (double)p.K * p.ksz * p.ksz * p.C;
                        L.flops += 2.0 * out_e * p.ksz * p.ksz * p.C; L.bytes += es * (in_e + out_e) + 4.0 * w_e;
                        break;
                    }
                    if (o.backend && o.kind != OP_SPLITK) {      // tensor-core problem: its own descriptor array (one descriptor, or one per output phase)
                        if (k == i) L.first = n_tc;
                        const int mode = o.kind == OP_CONV_FWD ? CONV_FWD : o.kind == OP_CONV_DGRAD ? CONV_DGRAD : CONV_WGRAD;
                        const int nd = conv_tc_count(o.conv, mode);
                        tc.resize((size_t)(n_tc + std::max(nd, 1)) * tcb);
                        if (!nd || conv_tc_fill(o.conv, mode, tc.data() + (size_t)n_tc * tcb) != nd) { ctx->err = "tensor map encoding failed"; return RESIST_ECUDA; }
                        for (int d = 0; d < nd; ++d) {
                            L.gx = std::max(L.gx, conv_tc_tiles(tc.data() + (size_t)(n_tc + d) * tcb));
                            L.max_elems = (long long)conv_tc_merge((size_t)L.max_elems, conv_tc_smem(tc.data() + (size_t)(n_tc + d) * tcb));
                        }
                        n_tc += nd; L.ndesc += nd;
                        const ConvProb& p = o.conv;
                        const double in_e = (double)p.N * p.H * p.W * p.C, out_e = (double)p.N * p.P * p.Q * p.K, w_e = (double)p.K * p.ksz * p.ksz * p.C;
                        L.flops += 2.0 * out_e * p.ksz * p.ksz * p.C;
                        if (o.kind == OP_CONV_WGRAD) L.bytes += es * (in_e + out_e) + 4.0 * w_e;
                        else L.bytes += es * (in_e + out_e + w_e + (p.add ? (o.kind == OP_CONV_FWD ? out_e : in_e) : 0.0));
                        break;
                    }
                    if (k == i) L.first = (int)conv.size();
                    if (o.patch_images) sites.push_back({0, (int)conv.size(), 0, 0, slot});
                    conv.push_back(o.conv);
                    const ConvProb& p = o.conv;
                    if (o.kind == OP_SPLITK) { L.max_elems = std::max<long long>(L.max_elems, (long long)p.M * p.Ncol);
                        L.bytes += 4.0 * p.M * p.Ncol * (p.splits + 1); }
                    else { L.gx = std::max(L.gx, p.tiles_m * p.tiles_n * p.splits);
                        const double in_e = (double)p.N * p.H * p.W * p.C, out_e = (double)p.N * p.P * p.Q * p.K, w_e = (double)p.K * p.ksz * p.ksz * p.C;
                        L.flops += 2.0 * out_e * p.ksz * p.ksz * p.C;
                        if (o.kind == OP_CONV_WGRAD) L.bytes += es * (in_e + out_e) + 4.0 * w_e;
                        else L.bytes += es * (in_e + out_e + w_e + (p.add ? (o.kind == OP_CONV_FWD ? out_e : in_e) : 0.0)); }
                    break; }
                case OP_BN_STATS: case OP_BN_APPLY: case OP_BN_BWD_REDUCE: case OP_BN_BWD_APPLY: case OP_BN_FWD_FUSED: case OP_BN_BWD_FUSED: case OP_BN_TILE_STATS: {
                    if (k == i) L.first = (int)bn.size();
                    bn.push_back(o.bn);
                    L.gx = std::max(L.gx, o.bn.chunks); L.max_c = std::max(L.max_c, o.bn.C);
                    L.max_elems = std::max<long long>(L.max_elems, o.bn.m * o.bn.C);
                    { const double e = (double)o.bn.m * o.bn.C;
                      if (o.kind == OP_BN_TILE_STATS) L.bytes += 8.0 * o.bn.chunks * o.bn.C;
                      else if (o.kind == OP_BN_STATS) L.bytes += o.bn.eval ? 0.0 : es * e;
                      else if (o.kind == OP_BN_APPLY) L.bytes += 2 * es * e;
                      else if (o.kind == OP_BN_BWD_REDUCE) L.bytes += 2 * es * e;
                      else if (o.kind == OP_BN_FWD_FUSED) L.bytes += 2 * es * e;          // x once from HBM (the second read is an L2 hit), a once
                      else if (o.kind == OP_BN_BWD_FUSED) L.bytes += es * e * (o.bn.add ? 4 : 3);
                      else L.bytes += es * e * (o.bn.add ? 4 : 3); }
                    break; }
                case OP_IM2COL: {
                    if (k == i) L.first = (int)col.size();
                    sites.push_back({2, (int)col.size(), 0, 0, slot});
                    col.push_back(o.col);
                    const double rows = (double)o.col.N * o.col.P * o.col.Q;
                    L.max_elems = std::max<long long>(L.max_elems, (long long)rows);
                    L.bytes += 2.0 * o.col.cols * rows + 2.0 * o.col.N * o.col.H * o.col.W * o.col.C;
                    break; }
                case OP_UPSAMPLE: {
                    if (k == i) L.first = (int)up.size();
                    up.push_back(o.up);
                    const double e = (double)o.up.N * o.up.K * 2.0;
                    L.max_elems = std::max<long long>(L.max_elems, (long long)o.up.N * o.up.H * o.up.W * (o.up.K / 8));
                    L.bytes += e * ((double)o.up.P * o.up.Q + (double)o.up.H * o.up.W);
                    break; }
                case OP_POOL_FWD: case OP_POOL_BWD: {
                    if (k == i) L.first = (int)pool.size();
                    pool.push_back(o.pool);
                    const PoolProb& p = o.pool;
                    L.max_elems = std::max<long long>(L.max_elems, (long long)p.N * (o.kind == OP_POOL_FWD ? p.P * p.Q : p.H * p.W) * p.C);
                    L.bytes += (double)p.N * p.C * (es * ((double)p.H * p.W + (double)p.P * p.Q) + 4.0 * p.P * p.Q);
                    break; }
                case OP_HEAD_FWD: case OP_HEAD_BWD: {
                    if (k == i) L.first = (int)head.size();
                    sites.push_back({1, (int)head.size(), 0, 1, slot});
                    if (o.kind == OP_HEAD_FWD) { sites.push_back({1, (int)head.size(), 1, 2, slot});
                        if (plan.sub == -2) { sites.push_back({1, (int)head.size(), 2, 3, 0}); sites.push_back({1, (int)head.size(), 3, 4, 0}); } }
                    head.push_back(o.head);
                    const HeadProb& p = o.head;
                    L.max_b = std::max(L.max_b, p.B); L.max_c = std::max(L.max_c, p.C); L.max_classes = std::max(L.max_classes, p.classes);
                    L.max_elems = std::max<long long>(L.max_elems, (long long)p.B * p.HW * p.C);
                    L.bytes += es * (double)p.B * p.HW * p.C + 4.0 * p.classes * p.C;
                    break; }
            }
        }
        // what a weight gradient in flight on the second stream reads, and whether this launch writes any of it
        {
            std::vector<const void*> wr; bool always = false;
            for (size_t k = i; k < j; ++k) {
                const Op& o = ops[k];
                switch (o.kind) {
                    case OP_CONV_FWD: case OP_CONV_DGRAD: wr.push_back(o.conv.out);
                        if (o.fuse == 1) wr.push_back(o.bn.a); else if (o.fuse == 2) wr.push_back(o.bn.dx);
                        break;
                    case OP_CONV_WGRAD: case OP_SPLITK: case OP_REPACK: break;
                    case OP_BN_STATS: case OP_BN_BWD_REDUCE: case OP_BN_TILE_STATS: break;
                    case OP_BN_APPLY: case OP_BN_FWD_FUSED: wr.push_back(o.bn.a); break;
                    case OP_BN_BWD_APPLY: case OP_BN_BWD_FUSED: wr.push_back(o.bn.dx); break;
                    default: always = true; break;
                }
            }
            L.join_before = false;
            if (L.kind == OP_CONV_WGRAD) { for (size_t k = i; k < j; ++k) { inflight.push_back(ops[k].conv.act); inflight.push_back(ops[k].conv.wgt); } }
            else if (L.kind != OP_SPLITK && L.kind != OP_REPACK && !inflight.empty()) {
                bool hit = always;
                for (const void* w : wr) for (const void* r : inflight) if (w == r) hit = true;
                if (hit) { L.join_before = true; inflight.clear(); }
            }
        }
        plan.launches.push_back(L);
        i = j;
    }
    // one device blob: conv | bn | pool | head | sites | sgd segments
    std::vector<Segment> segs; long long chunks = 0;
    if (plan.sub >= 0) held_segments(ctx, plan.sub, 1u << plan.sub, false, segs, chunks);
    else if (plan.sub == -1) for (int s = 0; s < ctx->S; ++s) held_segments(ctx, s, 1u << s, false, segs, chunks);
    size_t off = 0;
    const size_t o_conv = off; off += align_up(conv.size() * sizeof(ConvProb), 256);
    const size_t o_bn = off;   off += align_up(bn.size() * sizeof(BnProb), 256);
    const size_t o_pool = off; off += align_up(pool.size() * sizeof(PoolProb), 256);
    const size_t o_head = off; off += align_up(head.size() * sizeof(HeadProb), 256);
    const size_t o_site = off; off += align_up(sites.size() * sizeof(PatchSite), 256);
    const size_t o_seg = off;  off += align_up(segs.size() * sizeof(Segment), 256);
    const size_t o_tc = off;   off += align_up(tc.size(), 256);
    const size_t o_wtc = off;  off += align_up(wtc.size(), 256);
    const size_t o_up = off;   off += align_up(up.size() * sizeof(UpProb), 256);
    const size_t o_mm = off;   off += align_up(mm.size(), 256);
    const size_t o_col = off;  off += align_up(col.size() * sizeof(ColProb), 256);
    const size_t o_wmm = off;  off += align_up(wmm.size(), 256);
    ctx_free(ctx, plan.d_blob);
    plan.d_blob = ctx_alloc(ctx, off + 256); plan.blob_bytes = off;
    if (!plan.d_blob) { ctx->err = "allocator returned NULL for the launch plan"; return RESIST_ENOMEM; }
    char* base = (char*)plan.d_blob;
    plan.d_conv = (ConvProb*)(base + o_conv); plan.d_bn = (BnProb*)(base + o_bn); plan.d_pool = (PoolProb*)(base + o_pool);
    plan.d_col = (ColProb*)(base + o_col);
    plan.d_head = (HeadProb*)(base + o_head); plan.d_sites = (PatchSite*)(base + o_site); plan.d_sgd = (Segment*)(base + o_seg);
    std::vector<PatchSite> dsites;
    for (const HostSite& h : sites) {
        PatchSite s{}; s.what = h.what; s.sub = h.sub;
        if (h.arr == 0) s.where = (void**)&plan.d_conv[h.idx].act;
        else if (h.arr == 2) s.where = (void**)&plan.d_col[h.idx].src;
        else if (h.field == 0) s.where = (void**)&plan.d_head[h.idx].labels;
        else if (h.field == 1) s.where = (void**)&plan.d_head[h.idx].loss_user;
        else if (h.field == 2) s.where = (void**)&plan.d_head[h.idx].logits_user;
        else s.where = (void**)&plan.d_head[h.idx].correct;
        dsites.push_back(s);
    }
    std::vector<char> host(off, 0);
    if (!conv.empty()) memcpy(host.data() + o_conv, conv.data(), conv.size() * sizeof(ConvProb));
    if (!bn.empty()) memcpy(host.data() + o_bn, bn.data(), bn.size() * sizeof(BnProb));
    if (!pool.empty()) memcpy(host.data() + o_pool, pool.data(), pool.size() * sizeof(PoolProb));
    if (!head.empty()) memcpy(host.data() + o_head, head.data(), head.size() * sizeof(HeadProb));
    if (!dsites.empty()) memcpy(host.data() + o_site, dsites.data(), dsites.size() * sizeof(PatchSite));
    if (!segs.empty()) memcpy(host.data() + o_seg, segs.data(), segs.size() * sizeof(Segment));
    if (!tc.empty()) memcpy(host.data() + o_tc, tc.data(), tc.size());
    plan.d_tc = base + o_tc; plan.tc_stride = tcb;
    if (!wtc.empty()) memcpy(host.data() + o_wtc, wtc.data(), wtc.size());
    plan.d_wtc = base + o_wtc; plan.wtc_stride = wtcb;
    if (!up.empty()) memcpy(host.data() + o_up, up.data(), up.size() * sizeof(UpProb));
    if (!col.empty()) memcpy(host.data() + o_col, col.data(), col.size() * sizeof(ColProb));
    plan.d_up = (UpProb*)(base + o_up);
    if (!mm.empty()) memcpy(host.data() + o_mm, mm.data(), mm.size());
    if (!wmm.empty()) memcpy(host.data() + o_wmm, wmm.data(), wmm.size());
    plan.d_mm = base + o_mm; plan.mm_stride = mmb; plan.d_wmm = base + o_wmm; plan.wmm_stride = wmmb;
    cudaError_t e = cudaMemcpyAsync(plan.d_blob, host.data(), off, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { ctx->err = std::string("plan upload: ") + cudaGetErrorString(e); return RESIST_ECUDA; }
    plan.nsites = (int)dsites.size(); plan.n_sgd_seg = (int)segs.size(); plan.sgd_chunks = chunks;
    plan.sgd_params = 0; for (const Segment& sg : segs) plan.sgd_params += (double)sg.len;
    return RESIST_OK;
}

static int ensure_workspace(resist_ctx* ctx, int B, std::vector<Needs>& needs) {
    needs.resize(ctx->S);
    size_t slice = 0;
    for (int s = 0; s < ctx->S; ++s) { needs[s] = measure_subnet(ctx, s, s, present_of(ctx, s), B, false, 1.f); slice = std::max(slice, needs[s].total); }
    if (slice <= ctx->ws_slice && (size_t)ctx->S * ctx->ws_slice <= ctx->ws_bytes) return RESIST_OK;
    if (slice <= ctx->ws_slice) slice = ctx->ws_slice;
    slice = align_up(slice + slice / 16, 1 << 20);               // a little slack: partitions differ slightly in size
    cudaDeviceSynchronize();
    ctx_free(ctx, ctx->d_ws); ctx->d_ws = nullptr; ctx->ws_bytes = 0; ctx->ws_slice = 0;
    for (Plan& p : ctx->plans) p.valid = false;
    std::fill(ctx->logits_dev.begin(), ctx->logits_dev.end(), nullptr);      // they pointed into the workspace just released
    ctx->d_ws = ctx_alloc(ctx, slice * ctx->S);
    if (!ctx->d_ws) { ctx->err = "allocator returned NULL for the activation workspace"; return RESIST_ENOMEM; }
    ctx->ws_bytes = slice * ctx->S; ctx->ws_slice = slice;
    return RESIST_OK;
}

// sub >= 0: one sub-ResNet; sub == -1: all S grouped
static int build_plan(resist_ctx* ctx, Plan& plan, int sub, int B, cudaStream_t st) {
    std::vector<Needs> needs;
    int rc = ensure_workspace(ctx, B, needs);
    if (rc) return rc;
    std::vector<Op> ops; plan.info = resist_step_info{};
    const int s0 = sub >= 0 ? sub : 0, s1 = sub >= 0 ? sub + 1 : ctx->S;
    for (int s = s0; s < s1; ++s) {
        Builder bd{ctx, B, s, s, false, 0, (char*)ctx->d_ws + (size_t)s * ctx->ws_slice};
        bd.es = ctx->opts.dtype == RESIST_BF16 ? 2 : 4; bd.ops = &ops;
        bd.bn_partial_need = needs[s].bn_partial; bd.wgrad_partial_need = needs[s].wgrad_partial; bd.gbig = needs[s].gbig; bd.up_need = needs[s].up;
        const size_t used = unroll_subnet(ctx, bd, present_of(ctx, s), 1.f);
        if (used > ctx->ws_slice) { ctx->err = "internal: workspace slice too small"; return RESIST_EINVAL; }
        ctx->logits_dev[s] = bd.logits; ctx->logits_B[s] = B;
        plan.info.conv_flops += bd.flops; plan.info.tensor_core_convs += bd.n_tc; plan.info.cuda_core_convs += bd.n_cc;
    }
    plan.sub = sub;
    rc = upload_plan(ctx, plan, ops, sub >= 0, st);
    if (rc) return rc;
    plan.B = B; plan.generation = ctx->generation; plan.valid = true;
    plan.info.workspace_bytes = (int64_t)ctx->ws_bytes;
    return RESIST_OK;
}

static int run_plan(resist_ctx* ctx, Plan& plan, const PatchArgs& pa, bool update, float lr, cudaStream_t st) {
    const bool bf = ctx->opts.dtype == RESIST_BF16;
    long long n_launch = 0;
    Profiler& pf = ctx->prof;
    const cudaStream_t caller_st = st;
    const bool overlap = !pf.on && update;
    if (overlap && !ctx->main_stream) {
        int lo = 0, hi = 0; cudaDeviceGetStreamPriorityRange(&lo, &hi);      // hi: numerically lowest = greatest priority
        if (cudaStreamCreateWithPriority(&ctx->main_stream, cudaStreamNonBlocking, hi) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_enter, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_leave, cudaEventDisableTiming) != cudaSuccess) { ctx->err = "cannot create the main stream"; return RESIST_ECUDA; }
    }
    if (overlap) { cudaEventRecord(ctx->ev_enter, caller_st); cudaStreamWaitEvent(ctx->main_stream, ctx->ev_enter, 0); st = ctx->main_stream; }
    if (plan.nsites) { pf.begin(PK_PATCH, 1, 0, 0, st); patch_kernel<<<(plan.nsites + 63) / 64, 64, 0, st>>>(plan.d_sites, plan.nsites, pa); pf.end(st); ++n_launch; }
    // A layer's weight gradient and data gradient both read dy and are independent of each other: the weight gradients
    // (and their partial-sum reductions) go to a second stream, one after another, while the main stream carries on
    // down the network.  Gradient buffers are recycled, so a launch that writes a buffer which a weight gradient in
    // flight still reads first waits for the second stream (join_before, worked out when the plan was built).
    // Per-kernel profiling keeps everything on one stream.
    if (overlap && !ctx->side_stream) {
        if (cudaStreamCreateWithFlags(&ctx->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_side_done, cudaEventDisableTiming) != cudaSuccess) { ctx->err = "cannot create the second stream"; return RESIST_ECUDA; }
    }
    bool side_pending = false;
    const cudaStream_t main_st = st;
    OpKind prev_kind = OP_HEAD_FWD;
    for (const Launch& L : plan.launches) {
        // early start of a warp-MMA convolution: not behind the im2col pass that writes the stem's packed weights, not while profiling
        const bool pdl_ok = !pf.on && prev_kind != OP_IM2COL; prev_kind = L.kind;
        const bool on_side = overlap && (L.kind == OP_CONV_WGRAD || ((L.kind == OP_SPLITK || L.kind == OP_REPACK) && side_pending));
        if (on_side) {
            cudaEventRecord(ctx->ev_fork, main_st); cudaStreamWaitEvent(ctx->side_stream, ctx->ev_fork, 0);
            st = ctx->side_stream;
        } else {
            st = main_st;
            if (side_pending && L.join_before) { cudaStreamWaitEvent(main_st, ctx->ev_side_done, 0); side_pending = false; }
        }
        int pk = 0, nk = 1;
        switch (L.kind) {
            case OP_CONV_FWD: pk = (L.backend >= 1000 && ((L.backend - 1000) & MMA_BACKEND_FUSED)) ? PK_CONV_FWD_MMA_BN : L.backend >= 200 ? PK_CONV_FWD_MMA : L.backend ? PK_CONV_FWD_TC : PK_CONV_FWD_CC; break;
            case OP_CONV_DGRAD: pk = (L.backend >= 1000 && ((L.backend - 1000) & MMA_BACKEND_FUSED)) ? PK_CONV_DGRAD_MMA_BN : L.backend >= 200 ? PK_CONV_DGRAD_MMA : L.backend ? PK_CONV_DGRAD_TC : PK_CONV_DGRAD_CC; break;
            case OP_CONV_WGRAD: pk = L.backend >= 200 ? PK_CONV_WGRAD_MMA : L.backend ? PK_CONV_WGRAD_TC : PK_CONV_WGRAD_CC; break;
            case OP_SPLITK: case OP_REPACK: pk = PK_SPLITK; break;
            case OP_BN_STATS: pk = PK_BN_STATS; nk = 2; break;
            case OP_BN_APPLY: pk = PK_BN_APPLY; break;
            case OP_BN_BWD_REDUCE: pk = PK_BN_BWD_REDUCE; nk = 2; break;
            case OP_BN_BWD_APPLY: pk = PK_BN_BWD_APPLY; break;
            case OP_POOL_FWD: pk = PK_POOL_FWD; break;
            case OP_POOL_BWD: pk = PK_POOL_BWD; break;
            case OP_HEAD_FWD: pk = PK_HEAD_FWD; nk = 3; break;
            case OP_HEAD_BWD: pk = PK_HEAD_BWD; nk = 3; break;
            case OP_UPSAMPLE: pk = PK_UPSAMPLE; break;
            case OP_IM2COL: pk = PK_IM2COL; break;
            case OP_BN_FWD_FUSED: pk = PK_BN_FWD_FUSED; break;
            case OP_BN_TILE_STATS: pk = PK_BN_TILE_STATS; break;
            case OP_BN_BWD_FUSED: pk = PK_BN_BWD_FUSED; break;
        }
        pf.begin(pk, nk, L.bytes, L.flops, st, L.label);
        switch (L.kind) {
            case OP_CONV_FWD: case OP_CONV_DGRAD: case OP_CONV_WGRAD: {
                const int mode = L.kind == OP_CONV_FWD ? CONV_FWD : L.kind == OP_CONV_DGRAD ? CONV_DGRAD : CONV_WGRAD;
                if (L.backend >= 200 && mode == CONV_WGRAD) { launch_conv_wgrad_mma_probs((const char*)plan.d_wmm + (size_t)L.first * plan.wmm_stride, L.count, L.gx, (size_t)L.max_elems, L.max_b, L.backend - 200, st, pdl_ok); ++n_launch; }
                else if (L.backend >= 200) {
                    if (!launch_conv_mma_probs((const char*)plan.d_mm + (size_t)L.first * plan.mm_stride, L.count, L.gx, (size_t)L.max_elems, L.backend - 1000, st, pdl_ok)) {
                        ctx->err = "warp-MMA convolution launch failed"; cudaGetLastError(); return RESIST_ECUDA; }
                }
                else if (L.backend && mode == CONV_WGRAD) { launch_conv_wgrad_tc_probs((const char*)plan.d_wtc + (size_t)L.first * plan.wtc_stride, L.count, L.gx, (size_t)L.max_elems, L.max_b, st); ++n_launch; }
                else if (L.backend) launch_conv_tc_probs((const char*)plan.d_tc + (size_t)L.first * plan.tc_stride, L.ndesc, L.gx, (size_t)L.max_elems, st);
                else launch_conv_ref(plan.d_conv + L.first, L.count, L.gx, mode, bf, st);
                ++n_launch; break; }
            case OP_SPLITK: launch_splitk_reduce(plan.d_conv + L.first, L.count, (int)L.max_elems, st); ++n_launch; break;
            case OP_REPACK: launch_repack_rows(plan.d_conv + L.first, L.count, (int)L.max_elems, st); ++n_launch; break;
            case OP_BN_STATS: launch_bn_stats(plan.d_bn + L.first, L.count, L.gx, L.max_c, bf, st); n_launch += 2; break;
            case OP_BN_APPLY: launch_bn_apply(plan.d_bn + L.first, L.count, L.max_elems, bf, st); ++n_launch; break;
            case OP_BN_BWD_REDUCE: launch_bn_bwd_reduce(plan.d_bn + L.first, L.count, L.gx, L.max_c, bf, st); n_launch += 2; break;
            case OP_BN_BWD_APPLY: launch_bn_bwd_apply(plan.d_bn + L.first, L.count, L.max_elems, bf, st); ++n_launch; break;
            case OP_POOL_FWD: launch_maxpool_fwd(plan.d_pool + L.first, L.count, L.max_elems, bf, st); ++n_launch; break;
            case OP_POOL_BWD: launch_maxpool_bwd(plan.d_pool + L.first, L.count, L.max_elems, bf, st); ++n_launch; break;
            case OP_HEAD_FWD: launch_head_fwd(plan.d_head + L.first, L.count, L.max_b, L.max_c, L.max_classes, bf, st); n_launch += 3; break;
            case OP_HEAD_BWD: launch_head_bwd(plan.d_head + L.first, L.count, L.max_b, L.max_c, L.max_classes, L.max_elems, bf, st); n_launch += 3; break;
            case OP_UPSAMPLE: launch_zero_stuff(plan.d_up + L.first, L.count, L.max_elems, st); ++n_launch; break;
            case OP_IM2COL: launch_im2col(plan.d_col + L.first, L.count, L.max_elems, st); ++n_launch; break;
            case OP_BN_TILE_STATS: launch_bn_finalize_tiles(plan.d_bn + L.first, L.count, L.max_c, st); ++n_launch; break;
            case OP_BN_FWD_FUSED:
                if (launch_bn_fused(plan.d_bn + L.first, L.count, L.gx, 0, st)) ++n_launch;
                else { launch_bn_stats(plan.d_bn + L.first, L.count, L.gx, L.max_c, bf, st); launch_bn_apply(plan.d_bn + L.first, L.count, L.max_elems, bf, st); n_launch += 3; }
                break;
            case OP_BN_BWD_FUSED:
                if (launch_bn_fused(plan.d_bn + L.first, L.count, L.gx, 1, st)) ++n_launch;
                else { launch_bn_bwd_reduce(plan.d_bn + L.first, L.count, L.gx, L.max_c, bf, st); launch_bn_bwd_apply(plan.d_bn + L.first, L.count, L.max_elems, bf, st); n_launch += 3; }
                break;
        }
        pf.end(st);
        if (on_side) { cudaEventRecord(ctx->ev_side_done, ctx->side_stream); side_pending = true; }
    }
    st = main_st;
    if (side_pending) cudaStreamWaitEvent(main_st, ctx->ev_side_done, 0);
    if (update && plan.sgd_chunks) {
        pf.begin(PK_SGD, 1, (bf ? 22.0 : 20.0) * plan.sgd_params, 0, st);
        launch_sgd(plan.d_sgd, plan.n_sgd_seg, plan.sgd_chunks, ctx->pa, lr, ctx->opts.momentum, ctx->opts.weight_decay, bf, st);
        pf.end(st);
        ++n_launch;
    }
    if (overlap) { cudaEventRecord(ctx->ev_leave, st); cudaStreamWaitEvent(caller_st, ctx->ev_leave, 0); }
    pf.collect(st);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { ctx->err = std::string("launch failed: ") + cudaGetErrorString(e); return RESIST_ECUDA; }
    ctx->info = plan.info; ctx->info.kernel_launches = n_launch;
    return RESIST_OK;
}

}  // namespace resist

using namespace resist;

extern "C" {

int resist_local_step(resist_ctx* ctx, int32_t subnet, const void* images, const int32_t* labels, int32_t B, float lr,
                      float* loss_out, resist_stream stream) {
    if (!ctx) return RESIST_EINVAL;
    if (ctx->state < 1) { ctx->err = "local step before partition"; return RESIST_ESTATE; }
    if (ctx->state == 3) { ctx->err = "local step after aggregate: the working copies are stale until the next partition"; return RESIST_ESTATE; }
    if (subnet < 0 || subnet >= ctx->S) { ctx->err = "subnet out of range"; return RESIST_EINVAL; }
    if (!images || !labels || B < 2 || B > 1024) { ctx->err = "need images, labels and 2 <= B <= 1024"; return RESIST_EINVAL; }
    cudaStream_t st = (cudaStream_t)stream;
    Plan& plan = ctx->plans[subnet];
    if (!plan.valid || plan.B != B || plan.generation != ctx->generation) { int rc = build_plan(ctx, plan, subnet, B, st); if (rc) return rc; }
    PatchArgs pa{}; pa.images[0] = images; pa.labels[0] = labels; pa.loss_out = loss_out;
    int rc = run_plan(ctx, plan, pa, true, lr, st);
    if (rc == RESIST_OK) ctx->state = 2;
    return rc;
}

int resist_local_step_grouped(resist_ctx* ctx, const void* const* images, const int32_t* const* labels, int32_t B, float lr,
                              float* loss_out, resist_stream stream) {
    if (!ctx) return RESIST_EINVAL;
    if (ctx->state < 1) { ctx->err = "local step before partition"; return RESIST_ESTATE; }
    if (ctx->state == 3) { ctx->err = "local step after aggregate: the working copies are stale until the next partition"; return RESIST_ESTATE; }
    if (!images || !labels || B < 2 || B > 1024) { ctx->err = "need images, labels and 2 <= B <= 1024"; return RESIST_EINVAL; }
    PatchArgs pa{};
    for (int s = 0; s < ctx->S; ++s) { if (!images[s] || !labels[s]) { ctx->err = "null image or label pointer"; return RESIST_EINVAL; }
        pa.images[s] = images[s]; pa.labels[s] = labels[s]; }
    pa.loss_out = loss_out;
    cudaStream_t st = (cudaStream_t)stream;
    Plan& plan = ctx->plans[ctx->S_cap];
    if (!plan.valid || plan.B != B || plan.generation != ctx->generation) { int rc = build_plan(ctx, plan, -1, B, st); if (rc) return rc; }
    int rc = run_plan(ctx, plan, pa, true, lr, st);
    if (rc == RESIST_OK) ctx->state = 2;
    return rc;
}

int resist_eval(resist_ctx* ctx, const void* images, const int32_t* labels, int32_t B, float* logits_out, float* loss_out,
                int32_t* correct_out, resist_stream stream) {
    if (!ctx) return RESIST_EINVAL;
    if (!images || B < 1 || B > 1024) { ctx->err = "need images and 1 <= B <= 1024"; return RESIST_EINVAL; }
    cudaStream_t st = (cudaStream_t)stream;
    int rc = ensure_param_arrays(ctx, std::max(ctx->S_cap, 1));
    if (rc) return rc;
    const int copy = ctx->S_cap;                               // the evaluation copy sits after the working copies
    const int S = std::max(ctx->S, 1);
    // refresh the evaluation copy from the global parameters
    Segment sp{0, ctx->L.n_params, 0, 0u, copy}, sb{0, ctx->L.n_buffers, 0, 0u, copy};
    rc = ensure_seg_table(ctx, 2); if (rc) return rc;
    Segment both[2] = {sp, sb};
    cudaError_t e = cudaMemcpyAsync(ctx->d_seg, both, sizeof(both), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { ctx->err = cudaGetErrorString(e); return RESIST_ECUDA; }
    launch_scatter(ctx->d_seg, 1, (sp.len + SEG_CHUNK - 1) / SEG_CHUNK, ctx->pa, false, ctx->opts.dtype == RESIST_BF16, st);
    launch_scatter_buffers(ctx->d_seg + 1, 1, (sb.len + SEG_CHUNK - 1) / SEG_CHUNK, ctx->pa, st);
    cudaStreamSynchronize(st);
    Plan& plan = ctx->plans[ctx->S_cap + 1];
    if (!plan.valid || plan.B != B || plan.generation != (unsigned long long)S) {
        std::vector<char> all(ctx->arch.num_blocks, 1);
        Needs n = measure_subnet(ctx, 0, copy, all, B, true, 1.f / (float)S);
        if (n.total > ctx->eval_ws_bytes) {
            cudaDeviceSynchronize(); ctx_free(ctx, ctx->d_eval_ws);
            ctx->d_eval_ws = ctx_alloc(ctx, n.total); ctx->eval_ws_bytes = ctx->d_eval_ws ? n.total : 0;
            if (!ctx->d_eval_ws) { ctx->err = "allocator returned NULL for the evaluation workspace"; return RESIST_ENOMEM; }
        }
        std::vector<Op> ops;
        Builder bd{ctx, B, 0, copy, true, 0, (char*)ctx->d_eval_ws}; bd.es = ctx->opts.dtype == RESIST_BF16 ? 2 : 4; bd.ops = &ops;
        bd.bn_partial_need = n.bn_partial; bd.wgrad_partial_need = n.wgrad_partial; bd.gbig = n.gbig; bd.up_need = n.up;
        unroll_subnet(ctx, bd, all, 1.f / (float)S);
        plan.sub = -2;
        rc = upload_plan(ctx, plan, ops, true, st);
        if (rc) return rc;
        plan.B = B; plan.generation = (unsigned long long)S; plan.valid = true;
    }
    PatchArgs pa{}; pa.images[0] = images; pa.labels[0] = labels; pa.loss_out = loss_out; pa.logits_out = logits_out; pa.correct = correct_out;
    const resist_step_info keep = ctx->info;
    rc = run_plan(ctx, plan, pa, false, 0.f, st);
    ctx->info = keep;
    return rc;
}

}  // extern "C"
