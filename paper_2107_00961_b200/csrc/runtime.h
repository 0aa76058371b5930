// Host runtime of the ResIST library: context, parameter layout, per-round schedule and launch plans.
#pragma once
#include <cstdio>
#include <string>
#include <vector>
#include "../../include/resist.h"
#include "internal.h"

namespace resist {

struct BNRef { long long g, b, buf; int c; };                 // offsets of gamma, beta; running stats (mean, var)
struct ConvRef { long long w; int k, cin, cout, stride; };
struct BlockRef { BNRef bn[3]; ConvRef conv[3]; ConvRef proj; int nconv; long long begin, end, buf_begin, buf_end; };
struct Layout {
    ConvRef stem; BNRef stem_bn; std::vector<BlockRef> blk; BNRef final_bn;
    long long head_w, head_b; int head_c; long long n_params, n_buffers;
};
Layout make_layout(const resist_arch& a, const std::vector<resist_block>& blocks);

enum OpKind {
    OP_CONV_FWD, OP_CONV_DGRAD, OP_CONV_WGRAD, OP_SPLITK, OP_BN_STATS, OP_BN_APPLY, OP_BN_BWD_REDUCE, OP_BN_BWD_APPLY,
    OP_POOL_FWD, OP_POOL_BWD, OP_HEAD_FWD, OP_HEAD_BWD, OP_UPSAMPLE, OP_IM2COL, OP_BN_FWD_FUSED, OP_BN_BWD_FUSED, OP_BN_TILE_STATS, OP_REPACK
};

// One operation of one sub-ResNet, keyed so that equal keys of different sub-ResNets share a launch.
struct Op {
    long long key; OpKind kind; int sub;
    ConvProb conv; BnProb bn; PoolProb pool; HeadProb head; UpProb up; ColProb col;
    int backend;          // convolutions: 0 = CUDA cores, 1 = tensor cores
    int patch_images;     // conv.act must be replaced by the caller's image pointer
    int fuse;             // warp-MMA convolutions: 1 = `bn` is the BN+ReLU forward of the output, 2 = the BN+ReLU backward whose da is the output; it runs in the same launch
};

struct PatchSite { void** where; int what; int sub; };        // what: 0 images, 1 labels, 2 loss_out, 3 logits_out, 4 correct

struct Launch {
    OpKind kind; int backend; int first, count;               // range in the typed device array
    int ndesc;                                                // tcgen05 forward / dgrad: descriptors of the launch (a stride-2 dgrad has one per output phase)
    int gx; long long max_elems; int max_b, max_c, max_classes;
    double bytes, flops;                                      // algorithmic work of this launch
    bool join_before;                                         // the main stream first waits for the weight gradients in flight
    char label[40];                                           // shape of the launch's first problem, for the per-launch trace
};

enum ProfKind {
    PK_CONV_FWD_CC, PK_CONV_DGRAD_CC, PK_CONV_WGRAD_CC, PK_CONV_FWD_TC, PK_CONV_DGRAD_TC, PK_CONV_WGRAD_TC, PK_SPLITK,
    PK_BN_STATS, PK_BN_APPLY, PK_BN_BWD_REDUCE, PK_BN_BWD_APPLY, PK_POOL_FWD, PK_POOL_BWD, PK_HEAD_FWD, PK_HEAD_BWD,
    PK_SGD, PK_PATCH, PK_SCATTER, PK_AGGREGATE, PK_UPSAMPLE, PK_CONV_FWD_MMA, PK_CONV_DGRAD_MMA, PK_CONV_WGRAD_MMA, PK_IM2COL, PK_BN_FWD_FUSED, PK_BN_BWD_FUSED, PK_CONV_FWD_MMA_BN, PK_CONV_DGRAD_MMA_BN, PK_BN_TILE_STATS, PK_COUNT
};
constexpr double PROFILE_RIDGE = 250.0;          // FLOP per byte at which a B200's bf16 tensor peak meets its HBM bandwidth (about 1.63e15 / 6.5e12)
struct Profiler {
    bool on = false;
    std::vector<cudaEvent_t> pool; size_t used = 0;
    struct Pending { int kind; int launches; double bytes, flops; cudaEvent_t e0, e1; const char* label; };
    FILE* trace = nullptr;                                    // RESIST_LAUNCH_TRACE=<file>: one line per bracketed launch (label, ms, bytes, flops)
    std::vector<Pending> pending;
    // per family, split by what bounds the launch: [0] = HBM (arithmetic intensity of the launch's algorithmic work at or below
    // PROFILE_RIDGE FLOP per byte), [1] = tensor cores (above it)
    long long launches[PK_COUNT][2] = {}, ops[PK_COUNT][2] = {}; double ms[PK_COUNT][2] = {}, bytes[PK_COUNT][2] = {}, flops[PK_COUNT][2] = {};
    cudaEvent_t ev() { if (used == pool.size()) { cudaEvent_t e; cudaEventCreate(&e); pool.push_back(e); } return pool[used++]; }
    void begin(int kind, int launches_, double b, double f, cudaStream_t st, const char* label = "") {
        if (!on) return; Pending p{kind, launches_, b, f, ev(), ev(), label}; cudaEventRecord(p.e0, st); pending.push_back(p); }
    void end(cudaStream_t st) { if (!on) return; cudaEventRecord(pending.back().e1, st); }
    void collect(cudaStream_t st) {
        if (!on) return; cudaStreamSynchronize(st);
        for (auto& p : pending) { float t = 0.f; cudaEventElapsedTime(&t, p.e0, p.e1);
            const int b = p.flops > PROFILE_RIDGE * p.bytes ? 1 : 0;
            ms[p.kind][b] += t; launches[p.kind][b] += p.launches; ops[p.kind][b] += 1; bytes[p.kind][b] += p.bytes; flops[p.kind][b] += p.flops;
            if (trace) fprintf(trace, "%d\t%s\t%.6f\t%.0f\t%.0f\n", p.kind, p.label, t, p.bytes, p.flops); }
        if (trace) fflush(trace);
        pending.clear(); used = 0; }
};

struct Plan {
    bool valid = false; int B = 0; unsigned long long generation = 0; int sub = -1;   // sub = -1: all sub-ResNets grouped
    std::vector<Launch> launches;
    void* d_blob = nullptr; size_t blob_bytes = 0;            // descriptor arrays in one device allocation
    ConvProb* d_conv = nullptr; BnProb* d_bn = nullptr; PoolProb* d_pool = nullptr; HeadProb* d_head = nullptr; UpProb* d_up = nullptr; ColProb* d_col = nullptr;
    PatchSite* d_sites = nullptr; int nsites = 0;
    void* d_tc = nullptr; size_t tc_stride = 0;              // tensor-core convolution descriptors
    void* d_wtc = nullptr; size_t wtc_stride = 0;            // tensor-core wgrad descriptors
    void* d_mm = nullptr; size_t mm_stride = 0; void* d_wmm = nullptr; size_t wmm_stride = 0;   // warp-level MMA descriptors
    Segment* d_sgd = nullptr; int n_sgd_seg = 0; long long sgd_chunks = 0; double sgd_params = 0;
    resist_step_info info{};
};

struct SubMem {           // device tensors of one sub-ResNet for one batch size (offsets into the workspace)
    size_t bytes = 0;
};

}  // namespace resist

struct resist_ctx {
    resist_arch arch{}; std::vector<resist_block> blocks; resist_opts opts{};
    resist::Layout L;
    resist_allocator alloc{}; bool own_alloc = false;
    int S = 0, S_cap = 0;                                      // current and allocated number of sub-ResNets
    std::vector<uint32_t> mask;                                // member_mask of the current round
    int state = 0;                                             // 0 = initialised, 1 = partitioned, 2 = stepped, 3 = aggregated
    unsigned long long generation = 0;                         // bumped by every partition
    long long aggregate_calls = 0;                             // counts resist_aggregate calls for opts.bn_stat_period
    resist::ParamArrays pa{};                                  // arrays hold S_cap + 1 copies; the last is the evaluation copy
    void* d_param_blob = nullptr;
    // workspace: per sub-ResNet slices of one allocation
    void* d_ws = nullptr; size_t ws_bytes = 0; size_t ws_slice = 0;
    void* d_eval_ws = nullptr; size_t eval_ws_bytes = 0;
    std::vector<resist::Plan> plans;                           // [S_cap] single plans, [S_cap] = grouped, [S_cap+1] = eval
    resist::Segment* d_seg = nullptr; int seg_cap = 0;         // scratch table for scatter / aggregate
    std::vector<float*> logits_dev; std::vector<int> logits_B; // last logits per sub-ResNet (device pointers into ws)
    resist_step_info info{};
    resist::Profiler prof;
    int sm_count = 148;
    // weight gradients run beside the data gradient of the same layer on a second stream (created on first use)
    cudaStream_t side_stream = nullptr; cudaEvent_t ev_fork = nullptr, ev_side_done = nullptr;
    // while they overlap, the main chain of the step runs on a stream of the library's own with the highest priority
    // (forked from and joined to the caller's stream), so that its CTAs are placed before those of the weight gradients
    cudaStream_t main_stream = nullptr; cudaEvent_t ev_enter = nullptr, ev_leave = nullptr;
    std::string err;
};
