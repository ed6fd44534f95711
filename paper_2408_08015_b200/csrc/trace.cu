// Launch accounting: every kernel launch of the library passes through a LaunchScope, which
// counts it and, while a trace is active, brackets it with CUDA events on the launching stream.
#include <atomic>
#include <cstdio>
#include <mutex>
#include <vector>

#include "../../include/asteroid.h"
#include "kernels.h"

namespace ast {

namespace {
struct Rec {
    int kind;
    double bytes, flops;
    cudaEvent_t e0, e1;
};
std::mutex g_mu;
uint64_t g_launches = 0;
bool g_tracing = false;
std::vector<Rec> g_recs;
std::vector<cudaEvent_t> g_pool;

cudaEvent_t take_event() {
    cudaEvent_t e;
    if (!g_pool.empty()) {
        e = g_pool.back();
        g_pool.pop_back();
        return e;
    }
    cudaEventCreate(&e);
    return e;
}

const char* const kNames[K_KINDS] = {
    "conv_fwd_simt", "conv_bwd_data_simt", "conv_bwd_weight_simt", "reduce_splits", "dw_fwd", "dw_bwd_data", "dw_bwd_weight",
    "dw_bwd_weight_finish", "bn_stats", "bn_stats_finish", "bn_bwd_reduce", "bn_bwd_finish", "ew_add", "ew_relu_mask", "ew_sum",
    "gap_fwd", "gap_bwd", "accumulate", "sgd_step", "refresh_derived", "loss_mse", "loss_softmax_xent", "pw_fwd_tcgen05", "pw_bwd_data_tcgen05", "pw_bwd_weight_tcgen05", "conv3x3_fwd_tcgen05", "conv3x3_bwd_data_tcgen05", "conv3x3_bwd_weight_tcgen05", "dw_bwd_fused", "conv_im2col", "conv_pad_unpad", "silu", "squeeze_excite"};
}  // namespace

int sm_count() {
    static std::atomic<int> cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n <= 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cache[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

const char* kernel_name(int kind) { return (kind >= 0 && kind < K_KINDS) ? kNames[kind] : "?"; }
uint64_t launches() { return g_launches; }
bool tracing() { return g_tracing; }

LaunchScope::LaunchScope(int kind, double alg_bytes, double flops, cudaStream_t s) : slot(-1), st(s) {
    std::lock_guard<std::mutex> lk(g_mu);
    ++g_launches;
    if (g_tracing) {
        Rec r{kind, alg_bytes, flops, take_event(), take_event()};
        cudaEventRecord(r.e0, st);
        g_recs.push_back(r);
        slot = (int)g_recs.size() - 1;
    }
}

LaunchScope::~LaunchScope() {
    if (slot >= 0) {
        std::lock_guard<std::mutex> lk(g_mu);
        if (slot < (int)g_recs.size()) cudaEventRecord(g_recs[slot].e1, st);
    }
}

}  // namespace ast

using namespace ast;

extern "C" {

int asteroid_trace_start(void) {
    std::lock_guard<std::mutex> lk(g_mu);
    for (auto& r : g_recs) {
        g_pool.push_back(r.e0);
        g_pool.push_back(r.e1);
    }
    g_recs.clear();
    g_tracing = true;
    return AST_OK;
}

int asteroid_trace_stop(ast_kernel_stat* out, int capacity, int* n_out) {
    if (!out || !n_out || capacity < 1) return AST_ERR_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return AST_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_mu);
    g_tracing = false;
    std::vector<ast_kernel_stat> agg(K_KINDS);
    for (int k = 0; k < K_KINDS; ++k) {
        agg[k] = ast_kernel_stat{};
        snprintf(agg[k].name, sizeof agg[k].name, "%s", kernel_name(k));
    }
    for (auto& r : g_recs) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, r.e0, r.e1);
        ast_kernel_stat& a = agg[r.kind];
        a.launches++;
        a.total_ms += ms;
        a.alg_bytes += r.bytes;
        a.flops += r.flops;
        g_pool.push_back(r.e0);
        g_pool.push_back(r.e1);
    }
    g_recs.clear();
    int n = 0;
    for (int k = 0; k < K_KINDS && n < capacity; ++k)
        if (agg[k].launches) out[n++] = agg[k];
    *n_out = n;
    return AST_OK;
}

}  // extern "C"
