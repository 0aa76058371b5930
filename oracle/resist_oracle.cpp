// CPU oracle for the ResIST hot path (arXiv 2107.00961).  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-code-path implementation of what the paper defines: the layer-wise
// random partition of residual blocks into S sub-ResNets (Sec. 2.2), one local SGD step of a
// pre-activation sub-ResNet (Algorithm 1; block structure Sec. 2.1 and the caption of Fig. 2),
// the reassembly that averages every parameter over the sub-ResNets that held it (Sec. 2.3;
// Appendix B, definition of the aggregated weights), and evaluation of the reassembled
// network with the 1/S scaling of Sec. 2.6.  Only tests, the smoke check and the benchmark's
// CPU-baseline leg may call it.  It shares no code with the CUDA library.
//
// Every routine is a template on the storage type R (float or double); every sum is
// accumulated in double.  `quant` = 1 additionally rounds stored activations, activation
// gradients and the convolution's copy of the weights to bf16 (round to nearest even), the
// storage rule of the tensor-core path; `quant` = 0 is the plain definition.
//
// Parity unpinned by the paper: it prints no worked numeric example of a forward or backward
// pass.  The layer routines are pinned by finite differences, closed forms and library
// routines in the CPU tests instead.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#include <algorithm>

namespace {

// ---------------------------------------------------------------- splitmix64 (Steele et al. 2014)
struct SplitMix64 {
    uint64_t state;
    explicit SplitMix64(uint64_t seed) : state(seed) {}
    uint64_t next() {
        state += 0x9E3779B97F4A7C15ULL;
        uint64_t z = state;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
        return z ^ (z >> 31);
    }
};

// ---------------------------------------------------------------- architecture descriptor
struct Block { int kind, stage, cin, cmid, cout, stride, proj, part; };
struct Arch {
    int in_h, in_w, in_c, classes, stem_k, stem_stride, stem_cout, stem_bn, stem_pool, nb;
    std::vector<Block> blk;
};
Arch parse_arch(const int32_t* d) {
    Arch a;
    a.in_h = d[0]; a.in_w = d[1]; a.in_c = d[2]; a.classes = d[3]; a.stem_k = d[4];
    a.stem_stride = d[5]; a.stem_cout = d[6]; a.stem_bn = d[7]; a.stem_pool = d[8]; a.nb = d[9];
    for (int i = 0; i < a.nb; ++i) {
        const int32_t* b = d + 10 + 8 * i;
        a.blk.push_back(Block{b[0], b[1], b[2], b[3], b[4], b[5], b[6], b[7]});
    }
    return a;
}

// Offsets of every tensor in the flat parameter vector and of every BN in the buffer vector.
struct BNRef { int64_t g, b, buf; int c; };            // gamma, beta offsets; buffer offset (mean, then var)
struct ConvRef { int64_t w; int k, cin, cout, stride; };
struct BlockRef { BNRef bn[3]; ConvRef conv[3]; ConvRef proj; int nconv; int64_t begin, end, buf_begin, buf_end; };
struct Layout {
    ConvRef stem; BNRef stem_bn; std::vector<BlockRef> blk; BNRef final_bn;
    int64_t head_w, head_b; int head_c; int64_t n_params, n_buffers;
};
Layout make_layout(const Arch& a) {
    Layout L; int64_t off = 0, boff = 0;
    auto conv = [&](int k, int cin, int cout, int stride) {
        ConvRef c{off, k, cin, cout, stride}; off += (int64_t)cout * k * k * cin; return c; };
    auto bn = [&](int c) { BNRef r{off, off + c, boff, c}; off += 2 * c; boff += 2 * c; return r; };
    L.stem = conv(a.stem_k, a.in_c, a.stem_cout, a.stem_stride);
    L.stem_bn = BNRef{0, 0, 0, 0};
    if (a.stem_bn) L.stem_bn = bn(a.stem_cout);
    int c = a.stem_cout;
    for (const Block& b : a.blk) {
        BlockRef r; r.begin = off; r.buf_begin = boff;
        if (b.kind == 0) {
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
        if (b.proj) r.proj = conv(1, b.cin, b.cout, b.stride);
        r.end = off; r.buf_end = boff;
        L.blk.push_back(r);
        c = b.cout;
    }
    L.final_bn = bn(c);
    L.head_c = c;
    L.head_w = off; off += (int64_t)a.classes * c;
    L.head_b = off; off += a.classes;
    L.n_params = off; L.n_buffers = boff;
    return L;
}

// ---------------------------------------------------------------- storage rounding
inline float bf16_rne(float x) {
    uint32_t u; std::memcpy(&u, &x, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) return x;          // inf / nan unchanged
    u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    float y; std::memcpy(&y, &u, 4); return y;
}
template <class R> inline R store(double v, int quant) {
    return quant ? (R)bf16_rne((float)v) : (R)v;
}

// ---------------------------------------------------------------- layer primitives (NHWC, KRSC)
inline int out_dim(int h, int k, int stride) { int pad = (k - 1) / 2; return (h + 2 * pad - k) / stride + 1; }

// y[n,p,q,k] = scale * sum_{r,s,c} a[n, p*stride+r-pad, q*stride+s-pad, c] * w[k,r,s,c]  (+ add[n,p,q,k])
// (scale is 1 in training; evaluation scales the residual branch of partitioned blocks by 1/S, Sec. 2.6)
template <class R>
void conv_fwd(const R* a, const R* w, const R* add, R* y, int N, int H, int W, int C, int K, int k,
              int stride, int quant, double scale = 1.0) {
    const int pad = (k - 1) / 2, P = out_dim(H, k, stride), Q = out_dim(W, k, stride);
    for (int n = 0; n < N; ++n)
      for (int p = 0; p < P; ++p)
        for (int q = 0; q < Q; ++q)
          for (int o = 0; o < K; ++o) {
              double acc = 0.0;
              for (int r = 0; r < k; ++r) {
                  int h = p * stride + r - pad; if (h < 0 || h >= H) continue;
                  for (int s = 0; s < k; ++s) {
                      int x = q * stride + s - pad; if (x < 0 || x >= W) continue;
                      const R* ap = a + (((int64_t)n * H + h) * W + x) * C;
                      const R* wp = w + (((int64_t)o * k + r) * k + s) * C;
                      for (int c = 0; c < C; ++c) acc += (double)ap[c] * (double)wp[c];
                  }
              }
              int64_t oi = (((int64_t)n * P + p) * Q + q) * K + o;
              acc *= scale;
              if (add) acc += (double)add[oi];
              y[oi] = store<R>(acc, quant);
          }
}

// da[n,h,x,c] = sum over (p,q,r,s,k) with p*stride+r-pad = h, q*stride+s-pad = x of dy[n,p,q,k]*w[k,r,s,c]
// (+ add[n,h,x,c]).  Written as a gather over output positions so each da element is one sum.
template <class R>
void conv_dgrad(const R* dy, const R* w, const R* add, R* da, int N, int H, int W, int C, int K, int k,
                int stride, int quant) {
    const int pad = (k - 1) / 2, P = out_dim(H, k, stride), Q = out_dim(W, k, stride);
    std::vector<double> acc(C);
    for (int n = 0; n < N; ++n)
      for (int h = 0; h < H; ++h)
        for (int x = 0; x < W; ++x) {
            std::fill(acc.begin(), acc.end(), 0.0);
            for (int r = 0; r < k; ++r) {
                int ph = h + pad - r; if (ph < 0 || ph % stride) continue; int p = ph / stride; if (p >= P) continue;
                for (int s = 0; s < k; ++s) {
                    int qx = x + pad - s; if (qx < 0 || qx % stride) continue; int q = qx / stride; if (q >= Q) continue;
                    const R* dyp = dy + (((int64_t)n * P + p) * Q + q) * K;
                    for (int o = 0; o < K; ++o) {
                        const R* wp = w + (((int64_t)o * k + r) * k + s) * C;
                        double g = (double)dyp[o];
                        for (int c = 0; c < C; ++c) acc[c] += g * (double)wp[c];
                    }
                }
            }
            int64_t ai = (((int64_t)n * H + h) * W + x) * C;
            for (int c = 0; c < C; ++c) {
                double v = acc[c]; if (add) v += (double)add[ai + c];
                da[ai + c] = store<R>(v, quant);
            }
        }
}

// dw[k,r,s,c] = sum_{n,p,q} dy[n,p,q,k] * a[n, p*stride+r-pad, q*stride+s-pad, c]   (never rounded)
template <class R>
void conv_wgrad(const R* dy, const R* a, R* dw, int N, int H, int W, int C, int K, int k, int stride) {
    const int pad = (k - 1) / 2, P = out_dim(H, k, stride), Q = out_dim(W, k, stride);
    std::vector<double> acc((size_t)K * k * k * C, 0.0);
    for (int n = 0; n < N; ++n)
      for (int p = 0; p < P; ++p)
        for (int q = 0; q < Q; ++q) {
            const R* dyp = dy + (((int64_t)n * P + p) * Q + q) * K;
            for (int r = 0; r < k; ++r) {
                int h = p * stride + r - pad; if (h < 0 || h >= H) continue;
                for (int s = 0; s < k; ++s) {
                    int x = q * stride + s - pad; if (x < 0 || x >= W) continue;
                    const R* ap = a + (((int64_t)n * H + h) * W + x) * C;
                    for (int o = 0; o < K; ++o) {
                        double g = (double)dyp[o];
                        double* accp = acc.data() + (((int64_t)o * k + r) * k + s) * C;
                        for (int c = 0; c < C; ++c) accp[c] += g * (double)ap[c];
                    }
                }
            }
        }
    for (size_t i = 0; i < acc.size(); ++i) dw[i] = (R)acc[i];
}

// Batch normalisation, training mode, followed by ReLU.  Per channel over m = N*H*W elements:
// mean, biased variance (two passes), xhat = (x-mean)/sqrt(var+eps), a = max(0, gamma*xhat+beta).
// Running statistics: (1-mom)*old + mom*new, the variance entering as the unbiased estimate.
template <class R>
void bn_relu_fwd(const R* x, const R* gamma, const R* beta, R* a, double* mean, double* invstd,
                 R* run_mean, R* run_var, int64_t m, int C, double eps, double mom, int quant) {
    for (int c = 0; c < C; ++c) {
        double s = 0.0; for (int64_t i = 0; i < m; ++i) s += (double)x[i * C + c];
        double mu = s / (double)m;
        double v = 0.0; for (int64_t i = 0; i < m; ++i) { double d = (double)x[i * C + c] - mu; v += d * d; }
        double var = v / (double)m;
        mean[c] = mu; invstd[c] = 1.0 / std::sqrt(var + eps);
        if (run_mean) {
            double unb = (m > 1) ? v / (double)(m - 1) : var;
            run_mean[c] = (R)((1.0 - mom) * (double)run_mean[c] + mom * mu);
            run_var[c] = (R)((1.0 - mom) * (double)run_var[c] + mom * unb);
        }
    }
    for (int64_t i = 0; i < m; ++i)
        for (int c = 0; c < C; ++c) {
            double z = ((double)x[i * C + c] - mean[c]) * invstd[c] * (double)gamma[c] + (double)beta[c];
            a[i * C + c] = store<R>(z > 0.0 ? z : 0.0, quant);
        }
}

// Backward of the above.  dz = da where the pre-ReLU value was > 0, else 0;
// dbeta = sum dz; dgamma = sum dz*xhat; dx = gamma*invstd*(dz - dbeta/m - xhat*dgamma/m) (+ add).
template <class R>
void bn_relu_bwd(const R* da, const R* x, const R* gamma, const R* beta, const double* mean,
                 const double* invstd, const R* add, R* dx, R* dgamma, R* dbeta, int64_t m, int C, int quant) {
    std::vector<double> sg(C, 0.0), sb(C, 0.0);
    for (int64_t i = 0; i < m; ++i)
        for (int c = 0; c < C; ++c) {
            double xh = ((double)x[i * C + c] - mean[c]) * invstd[c];
            double z = xh * (double)gamma[c] + (double)beta[c];
            double dz = z > 0.0 ? (double)da[i * C + c] : 0.0;
            sb[c] += dz; sg[c] += dz * xh;
        }
    for (int c = 0; c < C; ++c) { dgamma[c] = (R)sg[c]; dbeta[c] = (R)sb[c]; }
    for (int64_t i = 0; i < m; ++i)
        for (int c = 0; c < C; ++c) {
            double xh = ((double)x[i * C + c] - mean[c]) * invstd[c];
            double z = xh * (double)gamma[c] + (double)beta[c];
            double dz = z > 0.0 ? (double)da[i * C + c] : 0.0;
            double v = (double)gamma[c] * invstd[c] * (dz - sb[c] / (double)m - xh * sg[c] / (double)m);
            if (add) v += (double)add[i * C + c];
            dx[i * C + c] = store<R>(v, quant);
        }
}

// Evaluation-mode BN + ReLU with the running statistics.
template <class R>
void bn_relu_eval(const R* x, const R* gamma, const R* beta, const R* run_mean, const R* run_var, R* a,
                  int64_t m, int C, double eps, int quant) {
    for (int64_t i = 0; i < m; ++i)
        for (int c = 0; c < C; ++c) {
            double z = ((double)x[i * C + c] - (double)run_mean[c]) / std::sqrt((double)run_var[c] + eps)
                       * (double)gamma[c] + (double)beta[c];
            a[i * C + c] = store<R>(z > 0.0 ? z : 0.0, quant);
        }
}

// 3x3 stride-2 max-pool, padding 1; padded positions never win.  argmax = first maximum in
// row-major window order (flat input index), used to route the gradient.
template <class R>
void maxpool_fwd(const R* x, R* y, int32_t* arg, int N, int H, int W, int C) {
    const int P = out_dim(H, 3, 2), Q = out_dim(W, 3, 2);
    for (int n = 0; n < N; ++n) for (int p = 0; p < P; ++p) for (int q = 0; q < Q; ++q) for (int c = 0; c < C; ++c) {
        bool have = false; R best = 0; int32_t bi = -1;
        for (int r = 0; r < 3; ++r) { int h = 2 * p + r - 1; if (h < 0 || h >= H) continue;
            for (int s = 0; s < 3; ++s) { int w = 2 * q + s - 1; if (w < 0 || w >= W) continue;
                R v = x[(((int64_t)n * H + h) * W + w) * C + c];
                if (!have || v > best) { have = true; best = v; bi = h * W + w; } } }
        int64_t oi = (((int64_t)n * P + p) * Q + q) * C + c;
        y[oi] = best; if (arg) arg[oi] = bi;
    }
}
template <class R>
void maxpool_bwd(const R* dy, const int32_t* arg, R* dx, int N, int H, int W, int C, int quant) {
    const int P = out_dim(H, 3, 2), Q = out_dim(W, 3, 2);
    std::vector<double> acc((size_t)N * H * W * C, 0.0);
    for (int n = 0; n < N; ++n) for (int p = 0; p < P; ++p) for (int q = 0; q < Q; ++q) for (int c = 0; c < C; ++c) {
        int64_t oi = (((int64_t)n * P + p) * Q + q) * C + c;
        acc[((int64_t)n * H * W + arg[oi]) * C + c] += (double)dy[oi];
    }
    for (size_t i = 0; i < acc.size(); ++i) dx[i] = store<R>(acc[i], quant);
}

}  // namespace

namespace {

// ---------------------------------------------------------------- one sub-ResNet, one minibatch
template <class R> using Vec = std::vector<R>;

template <class R>
struct BlockState {            // what the backward pass needs from the forward pass of one present block
    int H, W, Ho, Wo;          // input and output spatial size
    Vec<R> x, a1, y1, a2, y2, a3;
    std::vector<double> mean[3], invstd[3];
};

// Forward + backward (+ SGD-momentum update) of the sub-ResNet made of the blocks with present[b] != 0
// (Algorithm 1, the body of the local-iteration loop).  An absent block is the identity map
// (Appendix B: the block's term is multiplied by its mask M = 0).
// params/mom/buffers are full-size vectors in the global layout; absent blocks are not touched.
template <class R>
int run_step(const Arch& A, const Layout& L, const uint8_t* present, R* params, R* mom, R* buffers,
             const R* images, const int32_t* labels, int B, double lr, double mu, double wd, double eps,
             double bn_mom, int quant, int do_update, R* grads_out, R* logits_out, double* loss_out) {
    if (B < 2) return -1;
    Vec<R> wq;                                    // the convolutions' copy of the weights
    const R* cw = params;
    if (quant) { wq.assign(params, params + L.n_params); for (auto& v : wq) v = (R)bf16_rne((float)v); cw = wq.data(); }
    Vec<R> grads((size_t)L.n_params, (R)0);
    auto bnf = [&](const Vec<R>& x, const BNRef& r, Vec<R>& a, std::vector<double>& mean, std::vector<double>& invstd, int64_t m) {
        a.resize(x.size()); mean.resize(r.c); invstd.resize(r.c);
        bn_relu_fwd<R>(x.data(), params + r.g, params + r.b, a.data(), mean.data(), invstd.data(),
                       buffers ? buffers + r.buf : nullptr, buffers ? buffers + r.buf + r.c : nullptr, m, r.c, eps, bn_mom, quant);
    };
    auto bnb = [&](const Vec<R>& da, const Vec<R>& x, const BNRef& r, const std::vector<double>& mean,
                   const std::vector<double>& invstd, const R* add, Vec<R>& dx, int64_t m) {
        dx.resize(x.size());
        bn_relu_bwd<R>(da.data(), x.data(), params + r.g, params + r.b, mean.data(), invstd.data(), add, dx.data(),
                       grads.data() + r.g, grads.data() + r.b, m, r.c, quant);
    };

    // ---- stem
    int H = A.in_h, W = A.in_w;
    int Hs = out_dim(H, A.stem_k, A.stem_stride), Ws = out_dim(W, A.stem_k, A.stem_stride);
    Vec<R> stem_y((size_t)B * Hs * Ws * A.stem_cout), stem_a, stem_p;
    std::vector<double> stem_mean, stem_invstd; std::vector<int32_t> stem_arg;
    conv_fwd<R>(images, cw + L.stem.w, nullptr, stem_y.data(), B, H, W, A.in_c, A.stem_cout, A.stem_k, A.stem_stride, quant);
    Vec<R> cur = stem_y; int cH = Hs, cW = Ws, cC = A.stem_cout;
    if (A.stem_bn) { bnf(stem_y, L.stem_bn, stem_a, stem_mean, stem_invstd, (int64_t)B * Hs * Ws); cur = stem_a; }
    int Hp = cH, Wp = cW;
    if (A.stem_pool) {
        Hp = out_dim(cH, 3, 2); Wp = out_dim(cW, 3, 2);
        stem_p.resize((size_t)B * Hp * Wp * cC); stem_arg.resize(stem_p.size());
        maxpool_fwd<R>(cur.data(), stem_p.data(), stem_arg.data(), B, cH, cW, cC);
        cur = stem_p; cH = Hp; cW = Wp;
    }

    // ---- residual blocks, ascending network order
    std::vector<BlockState<R>> st(A.nb);
    for (int b = 0; b < A.nb; ++b) {
        if (!present[b]) continue;
        const Block& K = A.blk[b]; const BlockRef& r = L.blk[b]; BlockState<R>& s = st[b];
        s.H = cH; s.W = cW; s.Ho = out_dim(cH, 3, K.stride); s.Wo = out_dim(cW, 3, K.stride);
        const int64_t m_in = (int64_t)B * s.H * s.W, m_out = (int64_t)B * s.Ho * s.Wo;
        s.x = cur;
        bnf(s.x, r.bn[0], s.a1, s.mean[0], s.invstd[0], m_in);
        Vec<R> sc;
        const R* scp = s.x.data();                                   // identity skip reads the raw input
        if (K.proj) { sc.resize((size_t)m_out * K.cout);               // projection reads relu(bn1(x))
            conv_fwd<R>(s.a1.data(), cw + r.proj.w, nullptr, sc.data(), B, s.H, s.W, K.cin, K.cout, 1, K.stride, quant);
            scp = sc.data(); }
        Vec<R> out((size_t)m_out * K.cout);
        if (K.kind == 0) {
            s.y1.resize((size_t)m_out * K.cout);
            conv_fwd<R>(s.a1.data(), cw + r.conv[0].w, nullptr, s.y1.data(), B, s.H, s.W, K.cin, K.cout, 3, K.stride, quant);
            bnf(s.y1, r.bn[1], s.a2, s.mean[1], s.invstd[1], m_out);
            conv_fwd<R>(s.a2.data(), cw + r.conv[1].w, scp, out.data(), B, s.Ho, s.Wo, K.cout, K.cout, 3, 1, quant);
        } else {
            s.y1.resize((size_t)m_in * K.cmid);
            conv_fwd<R>(s.a1.data(), cw + r.conv[0].w, nullptr, s.y1.data(), B, s.H, s.W, K.cin, K.cmid, 1, 1, quant);
            bnf(s.y1, r.bn[1], s.a2, s.mean[1], s.invstd[1], m_in);
            s.y2.resize((size_t)m_out * K.cmid);
            conv_fwd<R>(s.a2.data(), cw + r.conv[1].w, nullptr, s.y2.data(), B, s.H, s.W, K.cmid, K.cmid, 3, K.stride, quant);
            bnf(s.y2, r.bn[2], s.a3, s.mean[2], s.invstd[2], m_out);
            conv_fwd<R>(s.a3.data(), cw + r.conv[2].w, scp, out.data(), B, s.Ho, s.Wo, K.cmid, K.cout, 1, 1, quant);
        }
        cur.swap(out); cH = s.Ho; cW = s.Wo; cC = K.cout;
    }

    // ---- final BN + ReLU, global average pool, linear head, mean softmax cross-entropy
    const int64_t mF = (int64_t)B * cH * cW; const int HW = cH * cW, NC = A.classes;
    Vec<R> xF = cur, aF; std::vector<double> meanF, invstdF;
    bnf(xF, L.final_bn, aF, meanF, invstdF, mF);
    Vec<R> pooled((size_t)B * cC), logits((size_t)B * NC), dlogits((size_t)B * NC);
    for (int n = 0; n < B; ++n) for (int c = 0; c < cC; ++c) {
        double s = 0.0; for (int i = 0; i < HW; ++i) s += (double)aF[((int64_t)n * HW + i) * cC + c];
        pooled[(size_t)n * cC + c] = (R)(s / HW);
    }
    double loss = 0.0;
    for (int n = 0; n < B; ++n) {
        for (int k = 0; k < NC; ++k) {
            double s = (double)params[L.head_b + k];
            for (int c = 0; c < cC; ++c) s += (double)params[L.head_w + (int64_t)k * cC + c] * (double)pooled[(size_t)n * cC + c];
            logits[(size_t)n * NC + k] = (R)s;
        }
        double mx = (double)logits[(size_t)n * NC]; for (int k = 1; k < NC; ++k) mx = std::max(mx, (double)logits[(size_t)n * NC + k]);
        double se = 0.0; for (int k = 0; k < NC; ++k) se += std::exp((double)logits[(size_t)n * NC + k] - mx);
        double lse = mx + std::log(se);
        loss += lse - (double)logits[(size_t)n * NC + labels[n]];
        for (int k = 0; k < NC; ++k)
            dlogits[(size_t)n * NC + k] = (R)((std::exp((double)logits[(size_t)n * NC + k] - lse) - (k == labels[n] ? 1.0 : 0.0)) / B);
    }
    loss /= B;
    if (loss_out) *loss_out = loss;
    if (logits_out) std::copy(logits.begin(), logits.end(), logits_out);

    // ---- backward: head, pool, final BN
    Vec<R> daF(aF.size());
    for (int k = 0; k < NC; ++k) {
        double sb = 0.0; for (int n = 0; n < B; ++n) sb += (double)dlogits[(size_t)n * NC + k];
        grads[L.head_b + k] = (R)sb;
        for (int c = 0; c < cC; ++c) {
            double s = 0.0; for (int n = 0; n < B; ++n) s += (double)dlogits[(size_t)n * NC + k] * (double)pooled[(size_t)n * cC + c];
            grads[L.head_w + (int64_t)k * cC + c] = (R)s;
        }
    }
    for (int n = 0; n < B; ++n) for (int c = 0; c < cC; ++c) {
        double s = 0.0; for (int k = 0; k < NC; ++k) s += (double)dlogits[(size_t)n * NC + k] * (double)params[L.head_w + (int64_t)k * cC + c];
        R g = store<R>(s / HW, quant);
        for (int i = 0; i < HW; ++i) daF[((int64_t)n * HW + i) * cC + c] = g;
    }
    Vec<R> dcur; bnb(daF, xF, L.final_bn, meanF, invstdF, nullptr, dcur, mF);

    // ---- backward through the present blocks, descending order
    for (int b = A.nb - 1; b >= 0; --b) {
        if (!present[b]) continue;
        const Block& K = A.blk[b]; const BlockRef& r = L.blk[b]; BlockState<R>& s = st[b];
        const int64_t m_in = (int64_t)B * s.H * s.W, m_out = (int64_t)B * s.Ho * s.Wo;
        const Vec<R>& dout = dcur;
        Vec<R> da1((size_t)m_in * K.cin), dsc_a1; const R* add_a1 = nullptr;
        if (K.proj) {
            conv_wgrad<R>(dout.data(), s.a1.data(), grads.data() + r.proj.w, B, s.H, s.W, K.cin, K.cout, 1, K.stride);
            dsc_a1.resize(da1.size());
            conv_dgrad<R>(dout.data(), cw + r.proj.w, nullptr, dsc_a1.data(), B, s.H, s.W, K.cin, K.cout, 1, K.stride, quant);
            add_a1 = dsc_a1.data();
        }
        if (K.kind == 0) {
            Vec<R> da2((size_t)m_out * K.cout), dy1;
            conv_wgrad<R>(dout.data(), s.a2.data(), grads.data() + r.conv[1].w, B, s.Ho, s.Wo, K.cout, K.cout, 3, 1);
            conv_dgrad<R>(dout.data(), cw + r.conv[1].w, nullptr, da2.data(), B, s.Ho, s.Wo, K.cout, K.cout, 3, 1, quant);
            bnb(da2, s.y1, r.bn[1], s.mean[1], s.invstd[1], nullptr, dy1, m_out);
            conv_wgrad<R>(dy1.data(), s.a1.data(), grads.data() + r.conv[0].w, B, s.H, s.W, K.cin, K.cout, 3, K.stride);
            conv_dgrad<R>(dy1.data(), cw + r.conv[0].w, add_a1, da1.data(), B, s.H, s.W, K.cin, K.cout, 3, K.stride, quant);
        } else {
            Vec<R> da3((size_t)m_out * K.cmid), dy2, da2((size_t)m_in * K.cmid), dy1;
            conv_wgrad<R>(dout.data(), s.a3.data(), grads.data() + r.conv[2].w, B, s.Ho, s.Wo, K.cmid, K.cout, 1, 1);
            conv_dgrad<R>(dout.data(), cw + r.conv[2].w, nullptr, da3.data(), B, s.Ho, s.Wo, K.cmid, K.cout, 1, 1, quant);
            bnb(da3, s.y2, r.bn[2], s.mean[2], s.invstd[2], nullptr, dy2, m_out);
            conv_wgrad<R>(dy2.data(), s.a2.data(), grads.data() + r.conv[1].w, B, s.H, s.W, K.cmid, K.cmid, 3, K.stride);
            conv_dgrad<R>(dy2.data(), cw + r.conv[1].w, nullptr, da2.data(), B, s.H, s.W, K.cmid, K.cmid, 3, K.stride, quant);
            bnb(da2, s.y1, r.bn[1], s.mean[1], s.invstd[1], nullptr, dy1, m_in);
            conv_wgrad<R>(dy1.data(), s.a1.data(), grads.data() + r.conv[0].w, B, s.H, s.W, K.cin, K.cmid, 1, 1);
            conv_dgrad<R>(dy1.data(), cw + r.conv[0].w, add_a1, da1.data(), B, s.H, s.W, K.cin, K.cmid, 1, 1, quant);
        }
        Vec<R> dx;   // identity skip: the block's input also receives dout directly
        bnb(da1, s.x, r.bn[0], s.mean[0], s.invstd[0], K.proj ? nullptr : dout.data(), dx, m_in);
        dcur.swap(dx);
    }

    // ---- backward through the stem (no input gradient is needed)
    if (A.stem_pool) { Vec<R> d((size_t)B * Hs * Ws * A.stem_cout);
        maxpool_bwd<R>(dcur.data(), stem_arg.data(), d.data(), B, Hs, Ws, A.stem_cout, quant); dcur.swap(d); }
    if (A.stem_bn) { Vec<R> d; bnb(dcur, stem_y, L.stem_bn, stem_mean, stem_invstd, nullptr, d, (int64_t)B * Hs * Ws); dcur.swap(d); }
    conv_wgrad<R>(dcur.data(), images, grads.data() + L.stem.w, B, H, W, A.in_c, A.stem_cout, A.stem_k, A.stem_stride);

    if (grads_out) std::copy(grads.begin(), grads.end(), grads_out);

    // ---- SGD with momentum on the parameters this sub-ResNet holds:  g += wd*w;  v = mu*v + g;  w -= lr*v
    if (do_update) {
        std::vector<uint8_t> held((size_t)L.n_params, 1);
        for (int b = 0; b < A.nb; ++b) if (!present[b]) std::fill(held.begin() + L.blk[b].begin, held.begin() + L.blk[b].end, 0);
        for (int64_t i = 0; i < L.n_params; ++i) {
            if (!held[i]) continue;
            R g = (R)((double)grads[i] + wd * (double)params[i]);
            R v = (R)(mu * (double)mom[i] + (double)g);
            mom[i] = v;
            params[i] = (R)((double)params[i] - lr * (double)v);
        }
    }
    return 0;
}

// Evaluation of the reassembled global network (Sec. 2.6): every block present, BN with running
// statistics, the residual branch of every partitionable block multiplied by 1/S.
template <class R>
int run_eval(const Arch& A, const Layout& L, const R* params, const R* buffers, int S, const R* images,
             const int32_t* labels, int B, double eps, int quant, R* logits_out, double* loss_out, int32_t* correct_out) {
    Vec<R> wq; const R* cw = params;
    if (quant) { wq.assign(params, params + L.n_params); for (auto& v : wq) v = (R)bf16_rne((float)v); cw = wq.data(); }
    auto bne = [&](const Vec<R>& x, const BNRef& r, Vec<R>& a, int64_t m) { a.resize(x.size());
        bn_relu_eval<R>(x.data(), params + r.g, params + r.b, buffers + r.buf, buffers + r.buf + r.c, a.data(), m, r.c, eps, quant); };
    int H = A.in_h, W = A.in_w;
    int cH = out_dim(H, A.stem_k, A.stem_stride), cW = out_dim(W, A.stem_k, A.stem_stride), cC = A.stem_cout;
    Vec<R> cur((size_t)B * cH * cW * cC);
    conv_fwd<R>(images, cw + L.stem.w, nullptr, cur.data(), B, H, W, A.in_c, cC, A.stem_k, A.stem_stride, quant);
    if (A.stem_bn) { Vec<R> a; bne(cur, L.stem_bn, a, (int64_t)B * cH * cW); cur.swap(a); }
    if (A.stem_pool) { int Hp = out_dim(cH, 3, 2), Wp = out_dim(cW, 3, 2); Vec<R> p((size_t)B * Hp * Wp * cC);
        maxpool_fwd<R>(cur.data(), p.data(), nullptr, B, cH, cW, cC); cur.swap(p); cH = Hp; cW = Wp; }
    for (int b = 0; b < A.nb; ++b) {
        const Block& K = A.blk[b]; const BlockRef& r = L.blk[b];
        const int Ho = out_dim(cH, 3, K.stride), Wo = out_dim(cW, 3, K.stride);
        const int64_t m_in = (int64_t)B * cH * cW, m_out = (int64_t)B * Ho * Wo;
        const double scale = K.part ? 1.0 / (double)S : 1.0;
        Vec<R> a1, sc, out((size_t)m_out * K.cout); bne(cur, r.bn[0], a1, m_in);
        const R* scp = cur.data();
        if (K.proj) { sc.resize(out.size());
            conv_fwd<R>(a1.data(), cw + r.proj.w, nullptr, sc.data(), B, cH, cW, K.cin, K.cout, 1, K.stride, quant); scp = sc.data(); }
        if (K.kind == 0) {
            Vec<R> y1((size_t)m_out * K.cout), a2;
            conv_fwd<R>(a1.data(), cw + r.conv[0].w, nullptr, y1.data(), B, cH, cW, K.cin, K.cout, 3, K.stride, quant);
            bne(y1, r.bn[1], a2, m_out);
            conv_fwd<R>(a2.data(), cw + r.conv[1].w, scp, out.data(), B, Ho, Wo, K.cout, K.cout, 3, 1, quant, scale);
        } else {
            Vec<R> y1((size_t)m_in * K.cmid), a2, y2((size_t)m_out * K.cmid), a3;
            conv_fwd<R>(a1.data(), cw + r.conv[0].w, nullptr, y1.data(), B, cH, cW, K.cin, K.cmid, 1, 1, quant);
            bne(y1, r.bn[1], a2, m_in);
            conv_fwd<R>(a2.data(), cw + r.conv[1].w, nullptr, y2.data(), B, cH, cW, K.cmid, K.cmid, 3, K.stride, quant);
            bne(y2, r.bn[2], a3, m_out);
            conv_fwd<R>(a3.data(), cw + r.conv[2].w, scp, out.data(), B, Ho, Wo, K.cmid, K.cout, 1, 1, quant, scale);
        }
        cur.swap(out); cH = Ho; cW = Wo; cC = K.cout;
    }
    Vec<R> aF; bne(cur, L.final_bn, aF, (int64_t)B * cH * cW);
    const int HW = cH * cW, NC = A.classes; double loss = 0.0; int correct = 0;
    std::vector<double> pooled(cC), lg(NC);
    for (int n = 0; n < B; ++n) {
        for (int c = 0; c < cC; ++c) { double s = 0.0; for (int i = 0; i < HW; ++i) s += (double)aF[((int64_t)n * HW + i) * cC + c];
            pooled[c] = (double)(R)(s / HW); }
        int best = 0;
        for (int k = 0; k < NC; ++k) { double s = (double)params[L.head_b + k];
            for (int c = 0; c < cC; ++c) s += (double)params[L.head_w + (int64_t)k * cC + c] * pooled[c];
            lg[k] = (double)(R)s; if (lg[k] > lg[best]) best = k;
            if (logits_out) logits_out[(size_t)n * NC + k] = (R)s; }
        double mx = lg[best], se = 0.0; for (int k = 0; k < NC; ++k) se += std::exp(lg[k] - mx);
        if (labels) { loss += mx + std::log(se) - lg[labels[n]]; correct += (best == labels[n]); }
    }
    if (loss_out) *loss_out = loss / B;
    if (correct_out) *correct_out = correct;
    return 0;
}

// Reassembly (Sec. 2.3; Appendix B: W^(h) = sum_v M_v^(h) W_v^(h) / sum_v M_v^(h)).  The mean over the
// owners is evaluated in the storage precision as  W_first + (sum_v (W_v - W_first)) / count,  owners
// taken in ascending sub-ResNet order: algebraically the same mean, and averaging identical copies
// is then the identity bit for bit for every count.  A single owner is copied without arithmetic.
// Applied alike to parameters and to BN running statistics.
template <class R>
void aggregate_range(const R* const* sub, int S, R* global, int64_t n, const uint32_t* mask_per_elem) {
    for (int64_t i = 0; i < n; ++i) {
        uint32_t m = mask_per_elem[i]; int cnt = 0; R first = 0, acc = 0;
        for (int s = 0; s < S; ++s) if (m >> s & 1u) {
            if (cnt == 0) first = sub[s][i]; else { R d = (R)(sub[s][i] - first); acc = (R)(acc + d); }
            ++cnt;
        }
        if (cnt == 0) continue;                       // held by nobody this round: the global value stands
        if (cnt == 1) { global[i] = first; continue; }
        R q = (R)(acc / (R)cnt);
        global[i] = (R)(first + q);
    }
}
template <class R>
int run_aggregate(const Arch& A, const Layout& L, const uint32_t* member_mask, int S, const R* const* sub_params,
                  const R* const* sub_buffers, R* global_params, R* global_buffers) {
    const uint32_t all = (S >= 32) ? 0xFFFFFFFFu : ((1u << S) - 1u);
    std::vector<uint32_t> pm((size_t)L.n_params, all), bm((size_t)L.n_buffers, all);
    for (int b = 0; b < A.nb; ++b) {
        std::fill(pm.begin() + L.blk[b].begin, pm.begin() + L.blk[b].end, member_mask[b]);
        std::fill(bm.begin() + L.blk[b].buf_begin, bm.begin() + L.blk[b].buf_end, member_mask[b]);
    }
    aggregate_range<R>(sub_params, S, global_params, L.n_params, pm.data());
    if (sub_buffers && global_buffers) aggregate_range<R>(sub_buffers, S, global_buffers, L.n_buffers, bm.data());
    return 0;
}

// subResNets(.) of Algorithm 1, Sec. 2.2: the indices of the partitionable blocks are randomly
// permuted (Fisher-Yates, from the end, j = next() mod (i+1)) and dealt round-robin: position j of
// the permutation goes to sub-ResNet j mod S.  Every other block is held by all S.
// min_depth > 0 (Sec. 2.6, "Subnetwork Depth"; the starred block of Fig. 1): a sub-ResNet holding
// fewer than min_depth partitioned blocks is topped up by walking the permutation cyclically from
// its start and taking blocks it does not hold yet.
int run_partition(const Arch& A, uint64_t round_seed, int S, int min_depth, uint32_t* member_mask) {
    if (S < 1 || S > 32) return -1;
    std::vector<int> ids;
    for (int b = 0; b < A.nb; ++b) if (A.blk[b].part) ids.push_back(b);
    const int P = (int)ids.size();
    if (P > 0 && S > P && min_depth <= 0) return -2;
    if (min_depth > P) return -3;
    SplitMix64 rng(round_seed);
    for (int i = P - 1; i >= 1; --i) { int j = (int)(rng.next() % (uint64_t)(i + 1)); std::swap(ids[i], ids[j]); }
    const uint32_t all = (S >= 32) ? 0xFFFFFFFFu : ((1u << S) - 1u);
    for (int b = 0; b < A.nb; ++b) member_mask[b] = A.blk[b].part ? 0u : all;
    std::vector<int> held(S, 0);
    for (int j = 0; j < P; ++j) { member_mask[ids[j]] |= 1u << (j % S); ++held[j % S]; }
    for (int s = 0; s < S; ++s)
        for (int j = 0; j < P && held[s] < min_depth; ++j)
            if (!(member_mask[ids[j]] >> s & 1u)) { member_mask[ids[j]] |= 1u << s; ++held[s]; }
    return 0;
}

}  // namespace

// ---------------------------------------------------------------- C entry points (for the tests' ctypes wrapper)
extern "C" {

void oracle_splitmix64(uint64_t seed, int64_t n, uint64_t* out) {
    SplitMix64 g(seed); for (int64_t i = 0; i < n; ++i) out[i] = g.next();
}

int oracle_param_count(const int32_t* arch, int64_t* n_params, int64_t* n_buffers) {
    Arch A = parse_arch(arch); Layout L = make_layout(A);
    *n_params = L.n_params; *n_buffers = L.n_buffers; return 0;
}

// [begin, end) of each block in the flat parameter vector and in the buffer vector: out[4*b .. 4*b+3]
int oracle_block_ranges(const int32_t* arch, int64_t* out) {
    Arch A = parse_arch(arch); Layout L = make_layout(A);
    for (int b = 0; b < A.nb; ++b) { out[4 * b] = L.blk[b].begin; out[4 * b + 1] = L.blk[b].end;
        out[4 * b + 2] = L.blk[b].buf_begin; out[4 * b + 3] = L.blk[b].buf_end; }
    return 0;
}

int oracle_partition(const int32_t* arch, uint64_t round_seed, int S, int min_depth, uint32_t* member_mask) {
    Arch A = parse_arch(arch); return run_partition(A, round_seed, S, min_depth, member_mask);
}

#define ORACLE_INSTANTIATE(SUF, R)                                                                              \
int oracle_step_##SUF(const int32_t* arch, const uint8_t* present, R* params, R* mom, R* buffers,               \
                      const R* images, const int32_t* labels, int B, double lr, double mu, double wd,           \
                      double eps, double bn_mom, int quant, int do_update, R* grads_out, R* logits_out,         \
                      double* loss_out) {                                                                       \
    Arch A = parse_arch(arch); Layout L = make_layout(A);                                                       \
    return run_step<R>(A, L, present, params, mom, buffers, images, labels, B, lr, mu, wd, eps, bn_mom, quant,  \
                       do_update, grads_out, logits_out, loss_out);                                             \
}                                                                                                               \
int oracle_eval_##SUF(const int32_t* arch, const R* params, const R* buffers, int S, const R* images,           \
                      const int32_t* labels, int B, double eps, int quant, R* logits_out, double* loss_out,     \
                      int32_t* correct_out) {                                                                   \
    Arch A = parse_arch(arch); Layout L = make_layout(A);                                                       \
    return run_eval<R>(A, L, params, buffers, S, images, labels, B, eps, quant, logits_out, loss_out, correct_out); \
}                                                                                                               \
int oracle_aggregate_##SUF(const int32_t* arch, const uint32_t* member_mask, int S, const R* const* sub_params, \
                           const R* const* sub_buffers, R* global_params, R* global_buffers) {                  \
    Arch A = parse_arch(arch); Layout L = make_layout(A);                                                       \
    return run_aggregate<R>(A, L, member_mask, S, sub_params, sub_buffers, global_params, global_buffers);      \
}                                                                                                               \
void oracle_conv_fwd_##SUF(const R* a, const R* w, const R* add, R* y, int N, int H, int W, int C, int K,       \
                           int k, int stride, int quant, double scale) {                                        \
    conv_fwd<R>(a, w, add, y, N, H, W, C, K, k, stride, quant, scale);                                          \
}                                                                                                               \
void oracle_conv_dgrad_##SUF(const R* dy, const R* w, const R* add, R* da, int N, int H, int W, int C, int K,   \
                             int k, int stride, int quant) {                                                    \
    conv_dgrad<R>(dy, w, add, da, N, H, W, C, K, k, stride, quant);                                             \
}                                                                                                               \
void oracle_conv_wgrad_##SUF(const R* dy, const R* a, R* dw, int N, int H, int W, int C, int K, int k,          \
                             int stride) {                                                                      \
    conv_wgrad<R>(dy, a, dw, N, H, W, C, K, k, stride);                                                         \
}                                                                                                               \
void oracle_bn_relu_fwd_##SUF(const R* x, const R* gamma, const R* beta, R* a, double* mean, double* invstd,    \
                              R* run_mean, R* run_var, int64_t m, int C, double eps, double mom, int quant) {   \
    bn_relu_fwd<R>(x, gamma, beta, a, mean, invstd, run_mean, run_var, m, C, eps, mom, quant);                  \
}                                                                                                               \
void oracle_bn_relu_bwd_##SUF(const R* da, const R* x, const R* gamma, const R* beta, const double* mean,       \
                              const double* invstd, const R* add, R* dx, R* dgamma, R* dbeta, int64_t m, int C, \
                              int quant) {                                                                      \
    bn_relu_bwd<R>(da, x, gamma, beta, mean, invstd, add, dx, dgamma, dbeta, m, C, quant);                      \
}                                                                                                               \
void oracle_maxpool_fwd_##SUF(const R* x, R* y, int32_t* arg, int N, int H, int W, int C) {                     \
    maxpool_fwd<R>(x, y, arg, N, H, W, C);                                                                      \
}                                                                                                               \
void oracle_maxpool_bwd_##SUF(const R* dy, const int32_t* arg, R* dx, int N, int H, int W, int C) {             \
    maxpool_bwd<R>(dy, arg, dx, N, H, W, C, 0);                                                                 \
}

ORACLE_INSTANTIATE(f32, float)
ORACLE_INSTANTIATE(f64, double)

}  // extern "C"
