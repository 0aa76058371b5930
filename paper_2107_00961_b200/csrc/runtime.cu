// Host side of the C boundary: context life cycle, the partition of Algorithm 1 (subResNets), the scatter
// of the global parameters into the working copies, the reassembly, and the parity taps.
// The launch plans of the local step live in plan.cu.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <algorithm>
#include "runtime.h"

using namespace resist;

static std::string g_init_error;

#define CK(call)                                                                                         \
    do { cudaError_t e_ = (call); if (e_ != cudaSuccess) {                                               \
        ctx->err = std::string(#call) + ": " + cudaGetErrorString(e_); return RESIST_ECUDA; } } while (0)

namespace resist {

Layout make_layout(const resist_arch& a, const std::vector<resist_block>& blocks) {
    Layout L; long long off = 0, boff = 0;
    auto conv = [&](int k, int cin, int cout, int stride) { ConvRef c{off, k, cin, cout, stride}; off += (long long)cout * k * k * cin; return c; };
    auto bn = [&](int c) { BNRef r{off, off + c, boff, c}; off += 2 * c; boff += 2 * c; return r; };
    L.stem = conv(a.stem_k, a.in_c, a.stem_cout, a.stem_stride);
    L.stem_bn = BNRef{0, 0, 0, 0};
    if (a.stem_bn_relu) L.stem_bn = bn(a.stem_cout);
    int c = a.stem_cout;
    for (const resist_block& b : blocks) {
        BlockRef r{}; r.begin = off; r.buf_begin = boff;
        if (b.kind == RESIST_BASIC) {
            r.nconv = 2;
            r.bn[0] = bn(b.cin);  r.conv[0] = conv(3, b.cin, b.cout, b.stride);
            r.bn[1] = bn(b.cout); r.conv[1] = conv(3, b.cout, b.cout, 1);
        } else {
            r.nconv = 3;
            r.bn[0] = bn(b.cin);  r.conv[0] = conv(1, b.cin, b.cmid, 1);
            r.bn[1] = bn(b.cmid); r.conv[1] = conv(3, b.cmid, b.cmid, b.stride);
            r.bn[2] = bn(b.cmid); r.conv[2] = conv(1, b.cmid, b.cout, 1);
        }
        r.proj = ConvRef{0, 0, 0, 0, 0};
        if (b.has_projection) r.proj = conv(1, b.cin, b.cout, b.stride);
        r.end = off; r.buf_end = boff;
        L.blk.push_back(r);
        c = b.cout;
    }
    L.final_bn = bn(c); L.head_c = c;
    L.head_w = off; off += (long long)a.classes * c;
    L.head_b = off; off += a.classes;
    L.n_params = off; L.n_buffers = boff;
    return L;
}

// splitmix64 (Steele, Lea, Flood 2014): the stream that drives the partition and the initialiser
struct Mix64 {
    uint64_t s;
    uint64_t next() {
        s += 0x9E3779B97F4A7C15ULL;
        uint64_t z = s;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
        return z ^ (z >> 31);
    }
    double uniform() { return (double)(next() >> 11) * (1.0 / 9007199254740992.0); }
};

void* ctx_alloc(resist_ctx* ctx, size_t bytes) {
    if (bytes == 0) bytes = 256;
    void* p = nullptr;
    if (ctx->own_alloc) { if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); p = nullptr; } }
    else p = ctx->alloc.alloc(ctx->alloc.user, bytes);
    return p;
}
void ctx_free(resist_ctx* ctx, void* p) {
    if (!p) return;
    if (ctx->own_alloc) cudaFree(p); else ctx->alloc.release(ctx->alloc.user, p);
}

void free_plan(resist_ctx* ctx, Plan& p);   // plan.cu
int conv_tc_read_status();                  // conv_tc.cu
int* conv_tc_status_word();

// after a synchronisation: did any bounded device-side wait give up?
static int device_status(resist_ctx* ctx) {
    const int v = conv_tc_read_status();
    if (v) { ctx->err = "a bounded device-side wait gave up (code " + std::to_string(v) + ")"; return RESIST_ETIMEOUT; }
    return RESIST_OK;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// (re)allocates the flat arrays for S_cap sub-ResNets plus the evaluation copy, keeping the global values
int ensure_param_arrays(resist_ctx* ctx, int S) {
    if (S <= ctx->S_cap && ctx->d_param_blob) return RESIST_OK;
    const long long n = ctx->L.n_params, nb = ctx->L.n_buffers;
    const long long np = (long long)align_up((size_t)n, 64), nbp = (long long)align_up((size_t)nb, 64);   // copies start 256-byte aligned
    const int copies = S + 1;
    const bool bf = ctx->opts.dtype == RESIST_BF16;
    size_t bytes = 0;
    const size_t o_w = bytes;  bytes += align_up((size_t)copies * np * 4, 256);
    const size_t o_v = bytes;  bytes += align_up((size_t)copies * np * 4, 256);
    const size_t o_g = bytes;  bytes += align_up((size_t)copies * np * 4, 256);
    const size_t o_wb = bytes; bytes += bf ? align_up((size_t)copies * np * 2, 256) : 0;
    const size_t o_b = bytes;  bytes += align_up((size_t)copies * nbp * 4, 256);
    char* blob = (char*)ctx_alloc(ctx, bytes);
    if (!blob) { ctx->err = "allocator returned NULL for the working copies"; return RESIST_ENOMEM; }
    if (cudaMemset(blob, 0, bytes) != cudaSuccess) { ctx->err = "cudaMemset failed"; return RESIST_ECUDA; }
    for (Plan& p : ctx->plans) free_plan(ctx, p);
    ctx->plans.clear(); ctx->plans.resize(S + 2);
    ctx_free(ctx, ctx->d_param_blob);
    ctx->d_param_blob = blob;
    ctx->pa.w = (float*)(blob + o_w); ctx->pa.v = (float*)(blob + o_v); ctx->pa.g = (float*)(blob + o_g);
    ctx->pa.wb = bf ? (__nv_bfloat16*)(blob + o_wb) : nullptr; ctx->pa.buf = (float*)(blob + o_b);
    ctx->pa.n = np; ctx->pa.nbuf = nbp;
    ctx->S_cap = S;
    ctx->logits_dev.assign(S + 1, nullptr); ctx->logits_B.assign(S + 1, 0);
    return RESIST_OK;
}

int ensure_seg_table(resist_ctx* ctx, int n) {
    if (n <= ctx->seg_cap) return RESIST_OK;
    ctx_free(ctx, ctx->d_seg);
    ctx->seg_cap = n + 64;
    ctx->d_seg = (Segment*)ctx_alloc(ctx, sizeof(Segment) * ctx->seg_cap);
    if (!ctx->d_seg) { ctx->seg_cap = 0; ctx->err = "allocator returned NULL for the segment table"; return RESIST_ENOMEM; }
    return RESIST_OK;
}

// Runs of parameters held by sub-ResNet `sub` (consecutive held blocks merge into one run).
void held_segments(const resist_ctx* ctx, int sub, uint32_t bit, bool buffers, std::vector<Segment>& out, long long& chunks) {
    const Layout& L = ctx->L;
    const long long total = buffers ? L.n_buffers : L.n_params;
    long long run = 0;
    auto flush = [&](long long end) {
        if (end > run) { Segment s{run, end - run, chunks, 0u, sub}; chunks += (s.len + SEG_CHUNK - 1) / SEG_CHUNK; out.push_back(s); }
    };
    for (size_t b = 0; b < L.blk.size(); ++b) {
        if (ctx->mask[b] & bit) continue;
        flush(buffers ? L.blk[b].buf_begin : L.blk[b].begin);
        run = buffers ? L.blk[b].buf_end : L.blk[b].end;
    }
    flush(total);
}

}  // namespace resist

extern "C" {

void resist_splitmix64(uint64_t seed, int64_t n, uint64_t* out) {
    Mix64 g{seed};
    for (int64_t i = 0; i < n; ++i) out[i] = g.next();
}

const char* resist_last_error(resist_ctx* ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

int resist_init(const resist_arch* arch, const resist_opts* opts, uint64_t seed, const resist_allocator* alloc,
                resist_ctx** out) {
    if (!arch || !opts || !out) { g_init_error = "null argument"; return RESIST_EINVAL; }
    *out = nullptr;
    auto bad = [&](const char* m) { g_init_error = m; return RESIST_EINVAL; };
    if (arch->num_blocks < 0 || (arch->num_blocks > 0 && !arch->blocks)) return bad("bad block list");
    if (arch->in_h < 1 || arch->in_w < 1 || arch->in_c < 1 || arch->classes < 1 || arch->classes > 65536) return bad("bad input shape or class count");
    if (arch->stem_k % 2 != 1 || arch->stem_k > 11 || arch->stem_stride < 1 || arch->stem_stride > 2 || arch->stem_cout < 1) return bad("bad stem");
    if (opts->dtype != RESIST_F32 && opts->dtype != RESIST_BF16) return bad("bad dtype");
    int c = arch->stem_cout;
    for (int i = 0; i < arch->num_blocks; ++i) {
        const resist_block& b = arch->blocks[i];
        if (b.kind != RESIST_BASIC && b.kind != RESIST_BOTTLENECK) return bad("bad block kind");
        if (b.cin != c || b.cout < 1 || b.cmid < 1 || (b.stride != 1 && b.stride != 2)) return bad("block channels or stride inconsistent");
        if (!b.has_projection && (b.stride != 1 || b.cin != b.cout)) return bad("identity skip needs stride 1 and cin == cout");
        if (b.kind == RESIST_BASIC && b.cmid != b.cout) return bad("basic block needs cmid == cout");
        c = b.cout;
    }
    int dev = 0; int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || count == 0) { cudaGetLastError(); g_init_error = "no CUDA device"; return RESIST_ECUDA; }
    cudaGetDevice(&dev);
    resist_ctx* ctx = new resist_ctx();
    ctx->arch = *arch; ctx->blocks.assign(arch->blocks, arch->blocks + arch->num_blocks); ctx->arch.blocks = nullptr;
    ctx->opts = *opts;
    if (alloc && alloc->alloc && alloc->release) { ctx->alloc = *alloc; ctx->own_alloc = false; } else ctx->own_alloc = true;
    cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, dev);
    ctx->L = make_layout(ctx->arch, ctx->blocks);
    ctx->mask.assign(arch->num_blocks, 1u);
    const Layout& L = ctx->L;
    const size_t gbytes = align_up((size_t)L.n_params * 4, 256) + align_up((size_t)L.n_buffers * 4, 256);
    char* g = (char*)ctx_alloc(ctx, gbytes);
    if (!g) { g_init_error = "allocator returned NULL for the global parameters"; delete ctx; return RESIST_ENOMEM; }
    ctx->pa.global = (float*)g; ctx->pa.global_buf = (float*)(g + align_up((size_t)L.n_params * 4, 256));

    // He-normal initialisation: one Box-Muller stream (cosine branch, then sine) consumed in flat order
    std::vector<float> p((size_t)L.n_params, 0.f), buf((size_t)L.n_buffers, 0.f);
    Mix64 rng{seed}; bool have = false; double spare = 0.0;
    auto normal = [&]() {
        if (have) { have = false; return spare; }
        double u1 = rng.uniform(), u2 = rng.uniform();
        double r = std::sqrt(-2.0 * std::log1p(-u1)), t = 2.0 * 3.14159265358979323846 * u2;
        spare = r * std::sin(t); have = true; return r * std::cos(t);
    };
    auto fill_conv = [&](const ConvRef& cr) { const double sd = std::sqrt(2.0 / ((double)cr.k * cr.k * cr.cin));
        const long long n = (long long)cr.cout * cr.k * cr.k * cr.cin; for (long long i = 0; i < n; ++i) p[cr.w + i] = (float)(normal() * sd); };
    auto fill_bn = [&](const BNRef& r) { for (int i = 0; i < r.c; ++i) { p[r.g + i] = 1.f; buf[r.buf + r.c + i] = 1.f; } };
    fill_conv(L.stem); if (arch->stem_bn_relu) fill_bn(L.stem_bn);
    for (const BlockRef& r : L.blk) { for (int i = 0; i < r.nconv; ++i) { fill_bn(r.bn[i]); fill_conv(r.conv[i]); } if (r.proj.k) fill_conv(r.proj); }
    fill_bn(L.final_bn);
    { const double sd = std::sqrt(2.0 / (double)L.head_c); for (long long i = 0; i < (long long)arch->classes * L.head_c; ++i) p[L.head_w + i] = (float)(normal() * sd); }
    cudaError_t e = cudaMemcpy(ctx->pa.global, p.data(), p.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->pa.global_buf, buf.data(), buf.size() * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { g_init_error = std::string("upload failed: ") + cudaGetErrorString(e); ctx_free(ctx, g); delete ctx; return RESIST_ECUDA; }
    *out = ctx;
    return RESIST_OK;
}

int resist_destroy(resist_ctx* ctx) {
    if (!ctx) return RESIST_EINVAL;
    cudaDeviceSynchronize();
    for (Plan& p : ctx->plans) free_plan(ctx, p);
    ctx_free(ctx, ctx->d_param_blob); ctx_free(ctx, ctx->pa.global); ctx_free(ctx, ctx->d_ws); ctx_free(ctx, ctx->d_eval_ws);
    ctx_free(ctx, ctx->d_seg);
    if (ctx->side_stream) { cudaStreamDestroy(ctx->side_stream); cudaEventDestroy(ctx->ev_fork); cudaEventDestroy(ctx->ev_side_done); }
    if (ctx->main_stream) { cudaStreamDestroy(ctx->main_stream); cudaEventDestroy(ctx->ev_enter); cudaEventDestroy(ctx->ev_leave); }
    delete ctx;
    return RESIST_OK;
}

int resist_param_count(resist_ctx* ctx, int64_t* n_params, int64_t* n_buffers) {
    if (!ctx) return RESIST_EINVAL;
    if (n_params) *n_params = ctx->L.n_params;
    if (n_buffers) *n_buffers = ctx->L.n_buffers;
    return RESIST_OK;
}

int resist_set_params(resist_ctx* ctx, const float* host_params, const float* host_buffers) {
    if (!ctx) return RESIST_EINVAL;
    CK(cudaDeviceSynchronize());
    if (host_params) CK(cudaMemcpy(ctx->pa.global, host_params, (size_t)ctx->L.n_params * 4, cudaMemcpyHostToDevice));
    if (host_buffers) CK(cudaMemcpy(ctx->pa.global_buf, host_buffers, (size_t)ctx->L.n_buffers * 4, cudaMemcpyHostToDevice));
    return RESIST_OK;
}

int resist_get_params(resist_ctx* ctx, int32_t subnet, float* host_params, float* host_buffers) {
    if (!ctx) return RESIST_EINVAL;
    if (subnet >= ctx->S || subnet < -1) { ctx->err = "subnet out of range"; return RESIST_EINVAL; }
    if (subnet >= 0 && ctx->state < 1) { ctx->err = "no partition yet"; return RESIST_ESTATE; }
    CK(cudaDeviceSynchronize());
    const float* p = subnet < 0 ? ctx->pa.global : ctx->pa.w + (long long)subnet * ctx->pa.n;
    const float* b = subnet < 0 ? ctx->pa.global_buf : ctx->pa.buf + (long long)subnet * ctx->pa.nbuf;
    if (host_params) CK(cudaMemcpy(host_params, p, (size_t)ctx->L.n_params * 4, cudaMemcpyDeviceToHost));
    if (host_buffers) CK(cudaMemcpy(host_buffers, b, (size_t)ctx->L.n_buffers * 4, cudaMemcpyDeviceToHost));
    return device_status(ctx);
}

int resist_get_grads(resist_ctx* ctx, int32_t subnet, float* host_grads) {
    if (!ctx || !host_grads) return RESIST_EINVAL;
    if (subnet < 0 || subnet >= ctx->S) { ctx->err = "subnet out of range"; return RESIST_EINVAL; }
    if (ctx->state < 2) { ctx->err = "no local step yet"; return RESIST_ESTATE; }
    CK(cudaDeviceSynchronize());
    CK(cudaMemcpy(host_grads, ctx->pa.g + (long long)subnet * ctx->pa.n, (size_t)ctx->L.n_params * 4, cudaMemcpyDeviceToHost));
    for (size_t b = 0; b < ctx->L.blk.size(); ++b)          // blocks this sub-ResNet does not hold have no gradient
        if (!(ctx->mask[b] >> subnet & 1u))
            std::fill(host_grads + ctx->L.blk[b].begin, host_grads + ctx->L.blk[b].end, 0.f);
    return device_status(ctx);
}

int resist_get_shadow(resist_ctx* ctx, int32_t subnet, uint16_t* host_bf16) {
    if (!ctx || !host_bf16) return RESIST_EINVAL;
    if (subnet < 0 || subnet >= ctx->S) { ctx->err = "subnet out of range"; return RESIST_EINVAL; }
    if (ctx->opts.dtype != RESIST_BF16 || !ctx->pa.wb) { ctx->err = "no bf16 copy in fp32 mode"; return RESIST_EUNSUPPORTED; }
    CK(cudaDeviceSynchronize());
    CK(cudaMemcpy(host_bf16, ctx->pa.wb + (long long)subnet * ctx->pa.n, (size_t)ctx->L.n_params * 2, cudaMemcpyDeviceToHost));
    return RESIST_OK;
}

int resist_get_logits(resist_ctx* ctx, int32_t subnet, float* host_logits) {
    if (!ctx || !host_logits) return RESIST_EINVAL;
    if (subnet < 0 || subnet >= ctx->S) { ctx->err = "subnet out of range"; return RESIST_EINVAL; }
    if (ctx->state < 2 || !ctx->logits_dev[subnet]) { ctx->err = "no local step yet"; return RESIST_ESTATE; }
    CK(cudaDeviceSynchronize());
    CK(cudaMemcpy(host_logits, ctx->logits_dev[subnet], (size_t)ctx->logits_B[subnet] * ctx->arch.classes * 4, cudaMemcpyDeviceToHost));
    return RESIST_OK;
}

int resist_get_step_info(resist_ctx* ctx, resist_step_info* out) {
    if (!ctx || !out) return RESIST_EINVAL;
    *out = ctx->info;
    return RESIST_OK;
}

static const char* const PK_NAMES[PK_COUNT] = {
    "conv_fwd_cuda_core", "conv_dgrad_cuda_core", "conv_wgrad_cuda_core", "conv_fwd_tcgen05", "conv_dgrad_tcgen05",
    "conv_wgrad_tcgen05", "wgrad_splitk_reduce", "bn_stats", "bn_apply_relu", "bn_bwd_reduce", "bn_bwd_apply", "maxpool_fwd",
    "maxpool_bwd", "head_fwd", "head_bwd", "sgd_momentum", "patch_pointers", "scatter", "aggregate", "zero_stuff_dy", "conv_fwd_mma", "conv_dgrad_mma", "conv_wgrad_mma", "im2col_stem", "bn_relu_fwd_fused", "bn_relu_bwd_fused", "conv_fwd_mma_bn", "conv_dgrad_mma_bn", "bn_stats_from_tiles"};

int resist_set_profiling(resist_ctx* ctx, int32_t on) {
    if (!ctx) return RESIST_EINVAL;
    ctx->prof.on = on != 0;
    // RESIST_LAUNCH_TRACE=<file>: while profiling, every bracketed launch also appends "family-index, shape label, ms, bytes, flops"
    if (on && !ctx->prof.trace) { const char* f = getenv("RESIST_LAUNCH_TRACE"); if (f && *f) ctx->prof.trace = fopen(f, "a"); }
    return RESIST_OK;
}

int resist_get_profile(resist_ctx* ctx, resist_profile_entry* out, int32_t cap, int32_t* n) {
    if (!ctx || !n) return RESIST_EINVAL;
    Profiler& pf = ctx->prof;
    int k = 0;
    for (int i = 0; i < PK_COUNT; ++i)
        for (int b = 0; b < 2; ++b) {
            if (!pf.ops[i][b]) continue;
            if (out && k < cap) { resist_profile_entry& e = out[k]; memset(&e, 0, sizeof(e));
                snprintf(e.name, sizeof(e.name), "%s%s", PK_NAMES[i], b ? "@tensor" : "");
                e.launches = pf.launches[i][b]; e.operations = pf.ops[i][b]; e.ms = pf.ms[i][b]; e.bytes = pf.bytes[i][b]; e.flops = pf.flops[i][b]; }
            ++k;
        }
    *n = k;
    for (int i = 0; i < PK_COUNT; ++i) for (int b = 0; b < 2; ++b) { pf.launches[i][b] = pf.ops[i][b] = 0; pf.ms[i][b] = pf.bytes[i][b] = pf.flops[i][b] = 0; }
    return RESIST_OK;
}

int resist_partition(resist_ctx* ctx, uint64_t round_seed, int32_t S, uint32_t* member_mask, resist_stream stream) {
    if (!ctx) return RESIST_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (S < 1 || S > RESIST_MAX_SUBNETS) { ctx->err = "S must be in 1..32"; return RESIST_EINVAL; }
    std::vector<int> ids;
    for (int b = 0; b < ctx->arch.num_blocks; ++b) if (ctx->blocks[b].partitionable) ids.push_back(b);
    const int P = (int)ids.size(), min_depth = ctx->opts.min_depth;
    if (P > 0 && S > P && min_depth <= 0) { ctx->err = "more sub-ResNets than partitionable blocks and no minimum depth"; return RESIST_EINVAL; }
    if (min_depth > P) { ctx->err = "minimum depth exceeds the number of partitionable blocks"; return RESIST_EINVAL; }
    // Fisher-Yates from the end, then round-robin deal (Sec. 2.2)
    Mix64 rng{round_seed};
    for (int i = P - 1; i >= 1; --i) { const int j = (int)(rng.next() % (uint64_t)(i + 1)); std::swap(ids[i], ids[j]); }
    const uint32_t all = S >= 32 ? 0xFFFFFFFFu : ((1u << S) - 1u);
    std::vector<uint32_t> mask(ctx->arch.num_blocks);
    for (int b = 0; b < ctx->arch.num_blocks; ++b) mask[b] = ctx->blocks[b].partitionable ? 0u : all;
    std::vector<int> held(S, 0);
    for (int j = 0; j < P; ++j) { mask[ids[j]] |= 1u << (j % S); ++held[j % S]; }
    for (int s = 0; s < S; ++s)                                // minimum depth: walk the permutation from its start
        for (int j = 0; j < P && held[s] < min_depth; ++j)
            if (!(mask[ids[j]] >> s & 1u)) { mask[ids[j]] |= 1u << s; ++held[s]; }

    int rc = ensure_param_arrays(ctx, S);
    if (rc) return rc;
    ctx->S = S; ctx->mask = mask; ctx->generation++;
    if (member_mask) std::copy(mask.begin(), mask.end(), member_mask);

    // scatter: global -> working copies of the blocks each sub-ResNet holds; momentum restarted
    std::vector<Segment> segs, bsegs; long long chunks = 0, bchunks = 0;
    for (int s = 0; s < S; ++s) { held_segments(ctx, s, 1u << s, false, segs, chunks); held_segments(ctx, s, 1u << s, true, bsegs, bchunks); }
    rc = ensure_seg_table(ctx, (int)(segs.size() + bsegs.size()));
    if (rc) return rc;
    CK(cudaMemcpyAsync(ctx->d_seg, segs.data(), segs.size() * sizeof(Segment), cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(ctx->d_seg + segs.size(), bsegs.data(), bsegs.size() * sizeof(Segment), cudaMemcpyHostToDevice, st));
    const bool restart = ctx->opts.momentum_policy == RESIST_MOMENTUM_RESTART || ctx->state == 0;
    double held_p = 0, heldb = 0; for (const Segment& g : segs) held_p += (double)g.len; for (const Segment& g : bsegs) heldb += (double)g.len;
    const bool bf = ctx->opts.dtype == RESIST_BF16;
    ctx->prof.begin(PK_SCATTER, 2, held_p * (4.0 + 4.0 + (restart ? 4.0 : 0.0) + (bf ? 2.0 : 0.0)) + heldb * 8.0, 0, st);
    launch_scatter(ctx->d_seg, (int)segs.size(), chunks, ctx->pa, restart, bf, st);
    launch_scatter_buffers(ctx->d_seg + segs.size(), (int)bsegs.size(), bchunks, ctx->pa, st);
    ctx->prof.end(st); ctx->prof.collect(st);
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(st));     // the host-side segment vectors die here
    ctx->state = 1;
    return RESIST_OK;
}

int resist_aggregate(resist_ctx* ctx, resist_stream stream) {
    if (!ctx) return RESIST_EINVAL;
    if (ctx->state < 1) { ctx->err = "aggregate before partition"; return RESIST_ESTATE; }
    cudaStream_t st = (cudaStream_t)stream;
    const Layout& L = ctx->L; const int S = ctx->S;
    const uint32_t all = S >= 32 ? 0xFFFFFFFFu : ((1u << S) - 1u);
    std::vector<Segment> segs, bsegs; long long chunks = 0, bchunks = 0;
    auto build = [&](bool buffers, std::vector<Segment>& out, long long& ch) {
        const long long total = buffers ? L.n_buffers : L.n_params;
        long long run = 0; uint32_t run_mask = all;
        auto flush = [&](long long end) { if (end > run) { Segment s{run, end - run, ch, run_mask, buffers ? 1 : 0}; ch += (s.len + AGG_CHUNK - 1) / AGG_CHUNK; out.push_back(s); } run = end; };
        for (size_t b = 0; b < L.blk.size(); ++b) {
            const long long bb = buffers ? L.blk[b].buf_begin : L.blk[b].begin, be = buffers ? L.blk[b].buf_end : L.blk[b].end;
            if (ctx->mask[b] == run_mask) continue;           // extends the current run (block ranges are contiguous)
            flush(bb); run_mask = ctx->mask[b]; (void)be;
        }
        // the tail after the last block (final BN, head) is shared by all
        if (!L.blk.empty() && run_mask != all) { flush(buffers ? L.blk.back().buf_end : L.blk.back().end); run_mask = all; }
        flush(total);
    };
    // BN running statistics: at every call, or at every bn_stat_period-th one (Sec. 5, ImageNet settings)
    const bool with_stats = ctx->opts.bn_stat_period <= 1 || (++ctx->aggregate_calls % ctx->opts.bn_stat_period) == 0;
    build(false, segs, chunks); bchunks = chunks; if (with_stats) build(true, bsegs, bchunks);   // one table, one launch: the statistics' chunks follow the parameters'
    segs.insert(segs.end(), bsegs.begin(), bsegs.end());
    int rc = ensure_seg_table(ctx, (int)segs.size());
    if (rc) return rc;
    CK(cudaMemcpyAsync(ctx->d_seg, segs.data(), segs.size() * sizeof(Segment), cudaMemcpyHostToDevice, st));
    double rd = 0, wr = 0;
    for (const Segment& g : segs) { rd += (double)g.len * __builtin_popcount(g.mask); wr += (double)g.len; }
    ctx->prof.begin(PK_AGGREGATE, 1, 4.0 * (rd + wr), 0, st);
    const AggArrays arr{ctx->pa.w, ctx->pa.buf, ctx->pa.n, ctx->pa.nbuf, ctx->pa.global, ctx->pa.global_buf};
    launch_aggregate(ctx->d_seg, (int)segs.size(), bchunks, arr, S, st);
    ctx->prof.end(st); ctx->prof.collect(st);
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(st));
    ctx->state = 3;                                            // the working copies are stale until the next partition
    return device_status(ctx);
}

// Test hook of the bounded-wait reporting: writes `code` into the status word the kernels' bounded waits write on expiry, so that
// the next call that synchronises reports RESIST_ETIMEOUT (no kernel has to give up for the mapping to be exercised).
int resist_debug_set_wait_status(int32_t code) {
    int* w = conv_tc_status_word();
    return w && cudaMemcpy(w, &code, 4, cudaMemcpyHostToDevice) == cudaSuccess ? RESIST_OK : RESIST_ECUDA;
}

}  // extern "C"
