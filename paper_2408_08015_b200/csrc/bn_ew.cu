// BatchNorm statistics / backward reductions, elementwise pieces (residual add, activation
// masks, materialisation of a stage output), global average pooling, gradient accumulation,
// the SGD-momentum update and the two loss heads.  All are bandwidth-bound passes over
// [pixels][channels] tensors; reductions are two-stage and deterministic (no float atomics).
#include "kernels.h"

namespace ast {
namespace {

// ------------------------------------------------------------------ per-channel reductions
// A block owns `cw` channel groups (V channels each) and a contiguous pixel range; thread
// (row, jl) walks the range with stride `rows`.  OP::acc adds one pixel's contribution to the
// thread's NACC*V accumulators.  Rows are combined through shared memory, blocks through
// partial[block_y][acc][c], summed in fixed order (in double) by the finishing kernel.
struct StatsOp {
    static constexpr int NACC = 2, NCTX = 1;     // context: the pivot (first pixel's value of each channel)
    const void* z;
    template <typename T, int V> __device__ __forceinline__ void init(int c0, float (*ctx)[V]) const { ld_raw_w<T, V>(z, (size_t)c0, ctx[0]); }
    static constexpr int NLD = 1;                // tensors read per pixel
    template <typename T> __device__ __forceinline__ void load(size_t e, Vec<T>* r) const { r[0].load(z, e / Vec<T>::N); }
    template <typename T, int V> __device__ __forceinline__ void acc_raw(size_t, const Vec<T>* r, const float (*ctx)[V], float (*a)[V]) const {
        float v[V];
        r[0].unpack(v);
        acc_vals<V>(v, ctx, a);
    }
    template <typename T, int V> __device__ __forceinline__ void acc(size_t e, const float (*ctx)[V], float (*a)[V]) const {
        float v[V];
        ld_raw_w<T, V>(z, e, v);
        acc_vals<V>(v, ctx, a);
    }
    template <int V> __device__ __forceinline__ void acc_vals(const float* v, const float (*ctx)[V], float (*a)[V]) const {
        if (V % 2 == 0) {
            // two channels per packed fp32 instruction
#pragma unroll
            for (int q = 0; q < V; q += 2) {
                const float2 d = __fadd2_rn(make_float2(v[q], v[q + 1]), make_float2(-ctx[0][q], -ctx[0][q + 1]));
                const float2 s1 = __fadd2_rn(make_float2(a[0][q], a[0][q + 1]), d);
                const float2 s2 = __ffma2_rn(d, d, make_float2(a[1][q], a[1][q + 1]));
                a[0][q] = s1.x; a[0][q + 1] = s1.y;
                a[1][q] = s2.x; a[1][q + 1] = s2.y;
            }
        } else {
#pragma unroll
            for (int q = 0; q < V; ++q) {
                float d = v[q] - ctx[0][q];
                a[0][q] += d;
                a[1][q] = fmaf(d, d, a[1][q]);
            }
        }
    }
};

// sums of dpre = dy*mask(pre) and of dpre*xhat; the per-channel coefficients live in registers.  The activation is a pair
// of bounds (ReLU6: 0..6, ReLU: 0..inf, none: -inf..inf) so that every storage type and activation runs one instruction
// stream; xhat = z*rstd - mean*rstd is one fused multiply-add.
struct BwdOp {
    static constexpr int NACC = 2, NCTX = 4;     // context: scale, shift, -mean*rstd, rstd
    GradSrc g;            // k1 unused here
    const float* mean;
    const float* rstd;
    float lo, hi;
    template <typename T, int V> __device__ __forceinline__ void init(int c0, float (*ctx)[V]) const {
#pragma unroll
        for (int q = 0; q < V; ++q) {
            ctx[0][q] = g.scale ? __ldg(g.scale + c0 + q) : 1.f;
            ctx[1][q] = g.scale ? __ldg(g.shift + c0 + q) : 0.f;
            ctx[3][q] = mean ? __ldg(rstd + c0 + q) : 0.f;
            ctx[2][q] = mean ? -__ldg(mean + c0 + q) * ctx[3][q] : 0.f;
        }
    }
    static constexpr int NLD = 2;
    template <typename T> __device__ __forceinline__ void load(size_t e, Vec<T>* r) const {
        r[0].load(g.dy, e / Vec<T>::N);
        if (g.act != ACT_NONE || mean) r[1].load(g.z, e / Vec<T>::N);
    }
    template <typename T, int V> __device__ __forceinline__ void acc_raw(size_t, const Vec<T>* r, const float (*ctx)[V], float (*a)[V]) const {
        float d[V], z[V];
        r[0].unpack(d);
        if (g.act != ACT_NONE || mean) r[1].unpack(z);
        acc_vals<V>(d, z, ctx, a);
    }
    template <typename T, int V> __device__ __forceinline__ void acc(size_t e, const float (*ctx)[V], float (*a)[V]) const {
        float d[V], z[V];
        ld_raw_w<T, V>(g.dy, e, d);
        if (g.act != ACT_NONE || mean) ld_raw_w<T, V>(g.z, e, z);
        acc_vals<V>(d, z, ctx, a);
    }
    template <int V> __device__ __forceinline__ void acc_vals(const float* d, const float* z, const float (*ctx)[V], float (*a)[V]) const {
        if (g.act != ACT_NONE || mean) {
            if (V % 2 == 0) {
#pragma unroll
                for (int q = 0; q < V; q += 2) {
                    const float2 z2 = make_float2(z[q], z[q + 1]);
                    const float2 pre = __ffma2_rn(z2, make_float2(ctx[0][q], ctx[0][q + 1]), make_float2(ctx[1][q], ctx[1][q + 1]));
                    const float2 xh = __ffma2_rn(z2, make_float2(ctx[3][q], ctx[3][q + 1]), make_float2(ctx[2][q], ctx[2][q + 1]));
                    const float2 dm = make_float2((pre.x > lo && pre.x < hi) ? d[q] : 0.f, (pre.y > lo && pre.y < hi) ? d[q + 1] : 0.f);
                    const float2 s1 = __fadd2_rn(make_float2(a[0][q], a[0][q + 1]), dm);
                    const float2 s2 = __ffma2_rn(dm, xh, make_float2(a[1][q], a[1][q + 1]));
                    a[0][q] = s1.x; a[0][q + 1] = s1.y;
                    a[1][q] = s2.x; a[1][q + 1] = s2.y;
                }
            } else {
#pragma unroll
                for (int q = 0; q < V; ++q) {
                    const float pre = fmaf(z[q], ctx[0][q], ctx[1][q]);
                    const float dm = (pre > lo && pre < hi) ? d[q] : 0.f;
                    a[0][q] += dm;
                    a[1][q] = fmaf(dm, fmaf(z[q], ctx[3][q], ctx[2][q]), a[1][q]);
                }
            }
        } else {
#pragma unroll
            for (int q = 0; q < V; ++q) a[0][q] += d[q];
        }
    }
};

// Backward of a residual add followed by ReLU, fused with the BatchNorm-backward sums of the one operand branch that ends in
// a BatchNorm without activation: dst = d * [out > 0] is stored, and its sums (of dst and of dst * xhat, xhat from the
// branch's raw conv output z) are taken from the same registers.
struct MaskBwdOp {
    static constexpr int NACC = 2, NCTX = 2, NLD = 3;     // context: -mean*rstd, rstd
    const void* d;        // gradient w.r.t. the ReLU's output
    const void* out;      // the ReLU's output (its sign is the mask)
    const void* z;        // raw conv output of the BatchNorm branch
    void* dst;            // gradient w.r.t. the sum (and, by alias, w.r.t. both operands)
    const float* mean;
    const float* rstd;
    template <typename T, int V> __device__ __forceinline__ void init(int c0, float (*ctx)[V]) const {
#pragma unroll
        for (int q = 0; q < V; ++q) {
            ctx[1][q] = __ldg(rstd + c0 + q);
            ctx[0][q] = -__ldg(mean + c0 + q) * ctx[1][q];
        }
    }
    template <typename T> __device__ __forceinline__ void load(size_t e, Vec<T>* r) const {
        r[0].load(d, e / Vec<T>::N);
        r[1].load(out, e / Vec<T>::N);
        r[2].load(z, e / Vec<T>::N);
    }
    template <typename T, int V> __device__ __forceinline__ void acc_raw(size_t e, const Vec<T>* r, const float (*ctx)[V], float (*a)[V]) const {
        float g[V], y[V], zz[V];
        r[0].unpack(g);
        r[1].unpack(y);
        r[2].unpack(zz);
#pragma unroll
        for (int q = 0; q < V; ++q) g[q] = y[q] > 0.f ? g[q] : 0.f;
        Vec<T> o;
        o.pack(g);
        o.store(dst, e / Vec<T>::N);
        // the sums are of the gradient as stored (after rounding), like every other producer's
        o.unpack(g);
#pragma unroll
        for (int q = 0; q < V; ++q) {
            a[0][q] += g[q];
            a[1][q] = fmaf(g[q], fmaf(zz[q], ctx[1][q], ctx[0][q]), a[1][q]);
        }
    }
    template <typename T, int V> __device__ __forceinline__ void acc(size_t e, const float (*ctx)[V], float (*a)[V]) const {
        Vec<T> r[3];
        load<T>(e, r);
        acc_raw<T, V>(e, r, ctx, a);
    }
};

template <typename T, int V, typename OP>
__global__ void __launch_bounds__(512) chan_reduce_kernel(OP op, size_t pixels, int c, int cw, int rows, size_t pix_per_block,
                                                          float* __restrict__ partial) {
    pdl_wait();
    pdl_launch();
    extern __shared__ float red[];
    const int cg = c / V;
    const int jl = threadIdx.x % cw, row = threadIdx.x / cw;
    const int j = blockIdx.x * cw + jl;
    const bool active = row < rows && j < cg;
    const int c0 = j * V;
    float a[OP::NACC][V];
#pragma unroll
    for (int t = 0; t < OP::NACC; ++t)
#pragma unroll
        for (int q = 0; q < V; ++q) a[t][q] = 0.f;
    if (active) {
        float ctx[OP::NCTX][V];
        op.template init<T, V>(c0, ctx);
        size_t pbeg = (size_t)blockIdx.y * pix_per_block, pend = min(pixels, pbeg + pix_per_block);
        size_t p = pbeg + row;
        if (V == Vec<T>::N) {
            // the loads of a batch of pixels (eight vectors per thread) are issued before any is used: with one block per SM
            // the bytes in flight come from each thread's own batch
            constexpr int U = 8 / OP::NLD;
            for (; p + (size_t)(U - 1) * rows < pend; p += (size_t)U * rows) {
                Vec<T> r[U][OP::NLD];
#pragma unroll
                for (int u = 0; u < U; ++u) op.template load<T>((p + (size_t)u * rows) * c + c0, r[u]);
#pragma unroll
                for (int u = 0; u < U; ++u) op.template acc_raw<T, V>((p + (size_t)u * rows) * c + c0, r[u], ctx, a);
            }
        }
        for (; p < pend; p += rows) op.template acc<T, V>(p * c + c0, ctx, a);
    }
    const int width = cw * V;
    for (int t = 0; t < OP::NACC; ++t) {
        if (row < rows) {
#pragma unroll
            for (int q = 0; q < V; ++q) red[row * width + jl * V + q] = a[t][q];
        }
        __syncthreads();
        for (int e = threadIdx.x; e < width; e += blockDim.x) {
            int ch = blockIdx.x * width + e;
            if (ch < c) {
                float s = 0.f;
                for (int r2 = 0; r2 < rows; ++r2) s += red[r2 * width + e];
                partial[((size_t)blockIdx.y * OP::NACC + t) * c + ch] = s;
            }
        }
        __syncthreads();
    }
}

struct ReducePlan {
    int V, cw, rows, gx;
    size_t by, ppb, smem;
};

ReducePlan plan_reduce(int dtype, size_t pixels, int c, int nacc, size_t scratch_floats) {
    ReducePlan p;
    int vmax = dtype == 0 ? 4 : 8;
    p.V = (c % vmax == 0) ? vmax : 1;
    int cg = c / p.V;
    p.cw = cg < 32 ? cg : 32;
    p.rows = 512 / p.cw;
    p.gx = (cg + p.cw - 1) / p.cw;
    size_t by = (sm_count() + p.gx - 1) / p.gx;            // one 512-thread block per SM: half the partials of two 256-thread blocks
    size_t max_by = (pixels + (size_t)p.rows * 4 - 1) / ((size_t)p.rows * 4);
    if (by > max_by) by = max_by;
    size_t cap = scratch_floats / ((size_t)nacc * c);
    if (by > cap) by = cap;
    if (by < 1) by = 1;
    p.ppb = (pixels + by - 1) / by;
    p.by = (pixels + p.ppb - 1) / p.ppb;
    p.smem = (size_t)p.rows * p.cw * p.V * sizeof(float);
    return p;
}

double esz(int dtype) { return dtype == 0 ? 4.0 : 2.0; }

template <typename OP>
void launch_reduce(int dtype, const ReducePlan& p, const OP& op, size_t pixels, int c, float* partial, int kind, double bytes, cudaStream_t st) {
    LaunchScope ls(kind, bytes + 8.0 * c * p.by, 4.0 * pixels * c, st);
    dim3 grid(p.gx, (unsigned)p.by);
    if (dtype == 0) {
        if (p.V == 1) launch_pdl(chan_reduce_kernel<float, 1, OP>, grid, 512, p.smem, st, op, pixels, c, p.cw, p.rows, p.ppb, partial);
        else launch_pdl(chan_reduce_kernel<float, 4, OP>, grid, 512, p.smem, st, op, pixels, c, p.cw, p.rows, p.ppb, partial);
    } else {
        if (p.V == 1) launch_pdl(chan_reduce_kernel<__nv_bfloat16, 1, OP>, grid, 512, p.smem, st, op, pixels, c, p.cw, p.rows, p.ppb, partial);
        else launch_pdl(chan_reduce_kernel<__nv_bfloat16, 8, OP>, grid, 512, p.smem, st, op, pixels, c, p.cw, p.rows, p.ppb, partial);
    }
}

// A block of 1024 threads finishes 32 channels: thread (bg, cl) sums the partials of blocks bg, bg+32, ...
// of channel cl (32 consecutive channels per load: coalesced), the eight sub-sums are combined in
// fixed order through shared memory, in double (the thirty-two sub-sums in index order).  Returns true in the thread that owns the channel.
__device__ __forceinline__ bool sum_partials(const float* __restrict__ partial, int blocks, int c, int& ch, double& s1, double& s2) {
    __shared__ double sh[2][32][32];
    const int cl = threadIdx.x & 31, bg = threadIdx.x >> 5;
    ch = blockIdx.x * 32 + cl;
    double a1 = 0.0, a2 = 0.0;
    if (ch < c) {
        // sixteen partials per round are loaded before any is added: the loads overlap, the order of
        // the additions stays fixed
        for (int b0 = bg; b0 < blocks; b0 += 32 * 16) {
            float v1[16], v2[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int b = b0 + 32 * u;
                const bool ok = b < blocks;
                v1[u] = ok ? partial[((size_t)b * 2 + 0) * c + ch] : 0.f;
                v2[u] = ok ? partial[((size_t)b * 2 + 1) * c + ch] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                a1 += v1[u];
                a2 += v2[u];
            }
        }
    }
    sh[0][bg][cl] = a1;
    sh[1][bg][cl] = a2;
    __syncthreads();
    if (bg != 0 || ch >= c) return false;
    s1 = 0.0;
    s2 = 0.0;
#pragma unroll
    for (int k = 0; k < 32; ++k) {
        s1 += sh[0][k][cl];
        s2 += sh[1][k][cl];
    }
    return true;
}

template <typename T>
__global__ void __launch_bounds__(1024) bn_stats_finish(const float* __restrict__ partial, int blocks, int c, const T* __restrict__ z, double count,
                                                       const float* __restrict__ gamma, const float* __restrict__ beta, float eps, float momentum,
                                                       BnFwdOut o) {
    pdl_wait();
    pdl_launch();
    // the owner thread's per-channel inputs are requested before the partials so that all of the
    // kernel's global loads overlap
    const int chp = blockIdx.x * 32 + (threadIdx.x & 31);
    const bool owner = (threadIdx.x >> 5) == 0 && chp < c;
    // pivot: the first pixel's value, or (z == nullptr: partials written by the producing kernel) the running mean
    // as it stands before this update
    const float rm = owner ? o.run_mean[chp] : 0.f, rv = owner ? o.run_var[chp] : 0.f;
    const float pv = owner ? (z ? to_f<T>(z[chp]) : rm) : 0.f, gm = owner ? gamma[chp] : 0.f, bt = owner ? beta[chp] : 0.f;
    int ch;
    double s1, s2;
    if (!sum_partials(partial, blocks, c, ch, s1, s2)) return;
    double pivot = pv;
    double m1 = s1 / count;
    double mean = pivot + m1;
    double var = s2 / count - m1 * m1;
    if (var < 0.0) var = 0.0;
    double rstd = 1.0 / sqrt(var + (double)eps);
    double sc = (double)gm * rstd;
    o.mean[ch] = (float)mean;
    o.rstd[ch] = (float)rstd;
    o.scale[ch] = (float)sc;
    o.shift[ch] = (float)((double)bt - mean * sc);
    double unbiased = count > 1.0 ? var * count / (count - 1.0) : var;
    o.run_mean[ch] = (float)((1.0 - momentum) * rm + momentum * mean);
    o.run_var[ch] = (float)((1.0 - momentum) * rv + momentum * unbiased);
}

__global__ void __launch_bounds__(1024) bn_bwd_finish(const float* __restrict__ partial, int blocks, int c, double count,
                                                     const float* __restrict__ mean, const float* __restrict__ rstd,
                                                     const float* __restrict__ gamma, BnBwdOut o) {
    pdl_wait();
    pdl_launch();
    const int chp = blockIdx.x * 32 + (threadIdx.x & 31);
    const bool owner = (threadIdx.x >> 5) == 0 && chp < c && o.dgamma != nullptr;
    const float pr = owner ? rstd[chp] : 0.f, pm = owner ? mean[chp] : 0.f, pg = owner ? gamma[chp] : 0.f;
    int ch;
    double s1, s2;
    if (!sum_partials(partial, blocks, c, ch, s1, s2)) return;
    o.dbeta[ch] = (float)s1;
    if (o.dgamma) {
        o.dgamma[ch] = (float)s2;
        double r = pr, m = pm;
        double k1 = (double)pg * r;
        o.k1[ch] = (float)k1;
        o.k2[ch] = (float)(k1 * (-s1 + s2 * m * r) / count);
        o.k3[ch] = (float)(-k1 * s2 * r / count);
    }
}

// ------------------------------------------------------------------ elementwise
template <typename T, int V>
__global__ void __launch_bounds__(256) ew_add_kernel(ValSrc a, ValSrc b, int act, size_t groups, int c, T* __restrict__ out, T* __restrict__ out2) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= groups) return;
    size_t e = i * V;
    int c0 = (int)(e % c);
    float x[V], y[V];
    ld_val_w<T, V>(a, e, c0, x);
    if (b.p) {
        ld_val_w<T, V>(b, e, c0, y);
#pragma unroll
        for (int q = 0; q < V; ++q) x[q] += y[q];
    }
#pragma unroll
    for (int q = 0; q < V; ++q) x[q] = apply_act(x[q], act);
    st_raw_w<T, V>(out, e, x);
    if (out2) st_raw_w<T, V>(out2, e, x);
}

// mode 0: dst = d * [out_val > 0];  mode 1: dst = a + b
template <typename T, int V>
__global__ void __launch_bounds__(256) ew_flat_kernel(int mode, const T* __restrict__ a, const T* __restrict__ b, size_t groups, T* __restrict__ dst) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= groups) return;
    float x[V], y[V];
    ld_raw_w<T, V>(a, i * V, x);
    ld_raw_w<T, V>(b, i * V, y);
#pragma unroll
    for (int q = 0; q < V; ++q) x[q] = mode == 0 ? (y[q] > 0.f ? x[q] : 0.f) : x[q] + y[q];
    st_raw_w<T, V>(dst, i * V, x);
}

// Stride-2 3x3 convs on the stride-1 tensor-core kernels.
// Backward: up[n][2*ho][2*wo][c] = dz[n][ho][wo][c] (formed on load), zero elsewhere on the hi x wi grid: the input
// gradient of the stride-2 conv is the stride-1 input gradient of `up`.
template <typename T, int V>
__global__ void __launch_bounds__(256) ew_upsample2_kernel(GradSrc d, int hi, int wi, int ho, int wo, int c, size_t groups, T* __restrict__ up) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= groups) return;
    const int cv = c / V;
    const int j = (int)(i % cv);
    size_t t = i / cv;
    const int v = (int)(t % wi);
    t /= wi;
    const int u = (int)(t % hi), n = (int)(t / hi);
    float f[V];
#pragma unroll
    for (int q = 0; q < V; ++q) f[q] = 0.f;
    if (!(u & 1) && !(v & 1) && (u >> 1) < ho && (v >> 1) < wo)
        ld_grad_w<T, V>(d, (((size_t)n * ho + (u >> 1)) * wo + (v >> 1)) * c + (size_t)j * V, j * V, f);
    st_raw_w<T, V>(up, i * V, f);
}
// Forward: z[n][ho][wo][c] = full[n][2*ho][2*wo][c], `full` the stride-1 output on the hi x wi grid.
template <typename T, int V>
__global__ void __launch_bounds__(256) ew_subsample2_kernel(const T* __restrict__ full, int hi, int wi, int ho, int wo, int c, size_t groups, T* __restrict__ z) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= groups) return;
    const int cv = c / V;
    const int j = (int)(i % cv);
    size_t t = i / cv;
    const int x = (int)(t % wo);
    t /= wo;
    const int y = (int)(t % ho), n = (int)(t / ho);
    float f[V];
    ld_raw_w<T, V>(full, (((size_t)n * hi + 2 * y) * wi + 2 * x) * c + (size_t)j * V, f);
    st_raw_w<T, V>(z, i * V, f);
}

template <typename T> __global__ void gap_fwd_kernel(ValSrc x, int n, int hw, int c, T* __restrict__ out) {
    pdl_wait();
    pdl_launch();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * c) return;
    int ch = i % c, s = i / c;
    float acc = 0.f;
    for (int p = 0; p < hw; ++p) acc += ld_val<T>(x, ((size_t)s * hw + p) * c + ch, ch);
    out[i] = from_f<T>(acc / (float)hw);
}

template <typename T> __global__ void gap_bwd_kernel(const T* __restrict__ da, int n, int hw, int c, const T* addend, T* dx) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)n * hw * c) return;
    int ch = (int)(i % c);
    int s = (int)(i / ((size_t)hw * c));
    float v = to_f<T>(da[(size_t)s * c + ch]) / (float)hw;
    if (addend) v += to_f<T>(addend[i]);
    dx[i] = from_f<T>(v);
}

// ------------------------------------------------------------------ parameters
__global__ void accumulate_kernel(float* __restrict__ G, const float* __restrict__ g, size_t n4, size_t n) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n4) {
        float4 a = reinterpret_cast<float4*>(G)[i];
        float4 b = reinterpret_cast<const float4*>(g)[i];
        a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        reinterpret_cast<float4*>(G)[i] = a;
    } else {
        size_t e = n4 * 4 + (i - n4);
        if (e < n) G[e] += g[e];
    }
}

__device__ __forceinline__ void sgd1(float& w, float& v, float& G, float inv_m, float lr, float mu) {
    float g = G * inv_m;
    v = fmaf(mu, v, g);
    w = fmaf(-lr, v, w);
    G = 0.f;
}

__global__ void sgd_step_kernel(float* __restrict__ w, float* __restrict__ v, float* __restrict__ G, size_t n4, size_t n, float inv_m, float lr,
                                float mu) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n4) {
        float4 a = reinterpret_cast<float4*>(w)[i], b = reinterpret_cast<float4*>(v)[i], c = reinterpret_cast<float4*>(G)[i];
        sgd1(a.x, b.x, c.x, inv_m, lr, mu);
        sgd1(a.y, b.y, c.y, inv_m, lr, mu);
        sgd1(a.z, b.z, c.z, inv_m, lr, mu);
        sgd1(a.w, b.w, c.w, inv_m, lr, mu);
        reinterpret_cast<float4*>(w)[i] = a;
        reinterpret_cast<float4*>(v)[i] = b;
        reinterpret_cast<float4*>(G)[i] = c;
    } else {
        size_t e = n4 * 4 + (i - n4);
        if (e < n) sgd1(w[e], v[e], G[e], inv_m, lr, mu);
    }
}

__global__ void refresh_kernel(const float* __restrict__ w, const int32_t* __restrict__ perm, float* __restrict__ d,
                               __nv_bfloat16* __restrict__ wb, __nv_bfloat16* __restrict__ wtb, size_t n) {
    // This kernel writes the derived weight copies that other kernels stage BEFORE their dependency wait.  It therefore
    // never releases its dependents early: without a launch_dependents the next kernel in the stream starts only when this
    // grid has completed and its stores are visible, and every later kernel is ordered behind that one.
    pdl_wait();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        float t = w[perm[i]];
        d[i] = t;
        if (wb) {
            wb[i] = __float2bfloat16_rn(w[i]);
            wtb[i] = __float2bfloat16_rn(t);
        }
    }
}

// ------------------------------------------------------------------ losses
constexpr int LOSS_MAX_BLOCKS = 1024;

__device__ __forceinline__ float block_sum(float v, float* sh) {
    v = warp_sum(v);
    int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0) sh[wid] = v;
    __syncthreads();
    float r = 0.f;
    if (wid == 0) {
        r = lane < (blockDim.x >> 5) ? sh[lane] : 0.f;
        r = warp_sum(r);
    }
    __syncthreads();
    return r;   // valid in warp 0
}

__device__ __forceinline__ float block_max(float v, float* sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0) sh[wid] = v;
    __syncthreads();
    float r = sh[0];
    for (int i = 1; i < (blockDim.x >> 5); ++i) r = fmaxf(r, sh[i]);
    __syncthreads();
    return r;
}

// The block that takes the last ticket sums the per-block partials in index order.
__device__ void finish_loss(float part, float* scratch, unsigned* ticket, int nparts, float scale, float* loss, float* sh) {
    __shared__ bool last;
    if (threadIdx.x == 0) {
        scratch[blockIdx.x] = part;
        __threadfence();
        unsigned t = atomicAdd(ticket, 1u);
        last = (t == (unsigned)nparts - 1);
    }
    __syncthreads();
    if (last) {
        __threadfence();
        float s = 0.f;
        for (int i = threadIdx.x; i < nparts; i += blockDim.x) s += *((volatile float*)scratch + i);
        s = block_sum(s, sh);
        if (threadIdx.x == 0) {
            *loss = s * scale;
            *ticket = 0;
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(256) mse_kernel(const T* __restrict__ y, const T* __restrict__ t, size_t n, T* __restrict__ dy, float* loss,
                                                  float* scratch, unsigned* ticket) {
    pdl_wait();
    pdl_launch();
    __shared__ float sh[32];
    float acc = 0.f;
    const float k = 2.f / (float)n;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float d = to_f<T>(y[i]) - to_f<T>(t[i]);
        acc = fmaf(d, d, acc);
        dy[i] = from_f<T>(d * k);
    }
    float part = block_sum(acc, sh);
    finish_loss(part, scratch, ticket, gridDim.x, 1.f / (float)n, loss, sh);
}

// Vector form (16-byte loads and stores, two vectors of each operand requested before either is used); elements past the
// last whole vector are taken by block 0.  The order of additions is fixed by the launch shape.
template <typename T>
__global__ void __launch_bounds__(256) mse_vec_kernel(const T* __restrict__ y, const T* __restrict__ t, size_t n, T* __restrict__ dy, float* loss,
                                                      float* scratch, unsigned* ticket) {
    pdl_wait();
    pdl_launch();
    __shared__ float sh[32];
    constexpr int V = Vec<T>::N;
    const size_t nv = n / V, stride = (size_t)gridDim.x * blockDim.x;
    const float k = 2.f / (float)n;
    float acc = 0.f;
    auto one = [&](const Vec<T>& a, const Vec<T>& b, size_t i) {
        float fa[V], fb[V];
        a.unpack(fa);
        b.unpack(fb);
#pragma unroll
        for (int q = 0; q < V; ++q) {
            const float d = fa[q] - fb[q];
            acc = fmaf(d, d, acc);
            fa[q] = d * k;
        }
        Vec<T> o;
        o.pack(fa);
        o.store(dy, i);
    };
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + stride < nv; i += 2 * stride) {
        Vec<T> a0, b0, a1, b1;
        a0.load(y, i);
        b0.load(t, i);
        a1.load(y, i + stride);
        b1.load(t, i + stride);
        one(a0, b0, i);
        one(a1, b1, i + stride);
    }
    for (; i < nv; i += stride) {
        Vec<T> a0, b0;
        a0.load(y, i);
        b0.load(t, i);
        one(a0, b0, i);
    }
    if (blockIdx.x == 0) {
        for (size_t e = nv * V + threadIdx.x; e < n; e += blockDim.x) {
            const float d = to_f<T>(y[e]) - to_f<T>(t[e]);
            acc = fmaf(d, d, acc);
            dy[e] = from_f<T>(d * k);
        }
    }
    float part = block_sum(acc, sh);
    finish_loss(part, scratch, ticket, gridDim.x, 1.f / (float)n, loss, sh);
}

template <typename T>
__global__ void __launch_bounds__(256) xent_kernel(const T* __restrict__ logits, const int32_t* __restrict__ labels, int rows, int classes,
                                                   T* __restrict__ dl, float* loss, float* scratch, unsigned* ticket) {
    pdl_wait();
    pdl_launch();
    __shared__ float sh[32];
    const int r = blockIdx.x;
    const T* lg = logits + (size_t)r * classes;
    float mx = -INFINITY;
    for (int j = threadIdx.x; j < classes; j += blockDim.x) mx = fmaxf(mx, to_f<T>(lg[j]));
    mx = block_max(mx, sh);
    float se = 0.f;
    for (int j = threadIdx.x; j < classes; j += blockDim.x) se += expf(to_f<T>(lg[j]) - mx);
    se = block_sum(se, sh);
    __shared__ float se_all;
    if (threadIdx.x == 0) se_all = se;
    __syncthreads();
    se = se_all;
    const int lab = labels[r];
    const float inv_rows = 1.f / (float)rows;
    for (int j = threadIdx.x; j < classes; j += blockDim.x) {
        float p = expf(to_f<T>(lg[j]) - mx) / se;
        dl[(size_t)r * classes + j] = from_f<T>((p - (j == lab ? 1.f : 0.f)) * inv_rows);
    }
    float part = logf(se) - (to_f<T>(lg[lab]) - mx);
    finish_loss(part, scratch, ticket, rows, inv_rows, loss, sh);
}

}  // namespace

// =================================================================== launchers
void bn_stats(int dtype, const void* z, size_t pixels, int c, const float* gamma, const float* beta, float eps, float momentum, float* scratch,
              size_t scratch_floats, const BnFwdOut& o, cudaStream_t st) {
    ReducePlan p = plan_reduce(dtype, pixels, c, 2, scratch_floats);
    StatsOp op{z};
    launch_reduce(dtype, p, op, pixels, c, scratch, K_BN_STATS, (double)pixels * c * esz(dtype), st);
    LaunchScope ls(K_BN_STATS_FINISH, 8.0 * c * (p.by + 4), 10.0 * c, st);
    if (dtype == 0)
        launch_pdl(bn_stats_finish<float>, (c + 31) / 32, 1024, 0, st, scratch, (int)p.by, c, (const float*)z, (double)pixels, gamma, beta, eps, momentum, o);
    else
        launch_pdl(bn_stats_finish<__nv_bfloat16>, (c + 31) / 32, 1024, 0, st, scratch, (int)p.by, c, (const __nv_bfloat16*)z, (double)pixels, gamma, beta, eps,
                                                                       momentum, o);
}

void bn_stats_finish_partials(const float* partial, int blocks, size_t pixels, int c, const float* gamma, const float* beta, float eps,
                              float momentum, const BnFwdOut& o, cudaStream_t st) {
    LaunchScope ls(K_BN_STATS_FINISH, 8.0 * c * (blocks + 4), 10.0 * c, st);
    launch_pdl(bn_stats_finish<float>, (c + 31) / 32, 1024, 0, st, partial, blocks, c, (const float*)nullptr, (double)pixels, gamma, beta, eps, momentum,
               o);
}

void bn_bwd_reduce(int dtype, const void* dy, const void* z, size_t pixels, int c, const float* scale, const float* shift, int act,
                   const float* mean, const float* rstd, const float* gamma, float* scratch, size_t scratch_floats, const BnBwdOut& o,
                   cudaStream_t st) {
    ReducePlan p = plan_reduce(dtype, pixels, c, 2, scratch_floats);
    BwdOp op{GradSrc{dy, z, scale, shift, nullptr, nullptr, nullptr, act}, mean, rstd, act == ACT_NONE ? -INFINITY : 0.f,
             act == ACT_RELU6 ? 6.f : INFINITY};
    launch_reduce(dtype, p, op, pixels, c, scratch, K_BN_BWD_REDUCE, (double)pixels * c * esz(dtype) * ((act != ACT_NONE || mean) ? 2.0 : 1.0), st);
    LaunchScope ls(K_BN_BWD_FINISH, 8.0 * c * (p.by + 4), 10.0 * c, st);
    launch_pdl(bn_bwd_finish, (c + 31) / 32, 1024, 0, st, scratch, (int)p.by, c, (double)pixels, mean, rstd, gamma, o);
}

bool ew_relu_mask_bn_sums(int dtype, const void* d, const void* out_val, const void* z, size_t pixels, int c, const float* mean, const float* rstd,
                          const float* gamma, void* dst, float* scratch, size_t scratch_floats, const BnBwdOut& o, cudaStream_t st) {
    if (c % (dtype == 0 ? 4 : 8)) return false;          // whole vectors per thread (the op stores what it loads)
    ReducePlan p = plan_reduce(dtype, pixels, c, 2, scratch_floats);
    MaskBwdOp op{d, out_val, z, dst, mean, rstd};
    launch_reduce(dtype, p, op, pixels, c, scratch, K_EW_MASK, (double)pixels * c * esz(dtype) * 4.0, st);
    LaunchScope ls(K_BN_BWD_FINISH, 8.0 * c * (p.by + 4), 10.0 * c, st);
    launch_pdl(bn_bwd_finish, (c + 31) / 32, 1024, 0, st, scratch, (int)p.by, c, (double)pixels, mean, rstd, gamma, o);
    return true;
}

void bn_bwd_finish_partials(const float* partial, int blocks, size_t pixels, int c, const float* mean, const float* rstd, const float* gamma,
                            const BnBwdOut& o, cudaStream_t st) {
    LaunchScope ls(K_BN_BWD_FINISH, 8.0 * c * (blocks + 4), 10.0 * c, st);
    launch_pdl(bn_bwd_finish, (c + 31) / 32, 1024, 0, st, partial, blocks, c, (double)pixels, mean, rstd, gamma, o);
}

// Vector form with the per-channel coefficients in registers: the grid's threads are cut to a multiple of the vectors per
// pixel, so that a thread striding by that count always lands on the same channels; four vectors of each operand are
// loaded before any is used.
template <typename T, int V>
__global__ void __launch_bounds__(256) ew_add_vec_kernel(ValSrc a, ValSrc b, int act, size_t groups, int vpr, size_t stride, T* __restrict__ out,
                                                          T* __restrict__ out2) {
    pdl_wait();
    pdl_launch();
    const size_t id = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= stride) return;
    const int c0 = (int)(id % (size_t)vpr) * V;
    float as[V], ah[V], bs[V], bh[V];
#pragma unroll
    for (int q = 0; q < V; ++q) {
        as[q] = a.scale ? __ldg(a.scale + c0 + q) : 1.f;
        ah[q] = a.scale ? __ldg(a.shift + c0 + q) : 0.f;
        bs[q] = (b.p && b.scale) ? __ldg(b.scale + c0 + q) : 1.f;
        bh[q] = (b.p && b.scale) ? __ldg(b.shift + c0 + q) : 0.f;
    }
    const float alo = a.act == ACT_NONE ? -INFINITY : 0.f, ahi = a.act == ACT_RELU6 ? 6.f : INFINITY;
    const float blo = b.act == ACT_NONE ? -INFINITY : 0.f, bhi = b.act == ACT_RELU6 ? 6.f : INFINITY;
    const float olo = act == ACT_NONE ? -INFINITY : 0.f, ohi = act == ACT_RELU6 ? 6.f : INFINITY;
    constexpr int U = 4;
    for (size_t i0 = id; i0 < groups; i0 += U * stride) {
        Vec<T> va[U], vb[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = i0 + u * stride;
            if (i < groups) {
                va[u].load(a.p, i);
                if (b.p) vb[u].load(b.p, i);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t i = i0 + u * stride;
            if (i < groups) {
                float x[V], y[V];
                va[u].unpack(x);
#pragma unroll
                for (int q = 0; q < V; ++q) x[q] = fminf(fmaxf(fmaf(x[q], as[q], ah[q]), alo), ahi);
                if (b.p) {
                    vb[u].unpack(y);
#pragma unroll
                    for (int q = 0; q < V; ++q) x[q] += fminf(fmaxf(fmaf(y[q], bs[q], bh[q]), blo), bhi);
                }
#pragma unroll
                for (int q = 0; q < V; ++q) x[q] = fminf(fmaxf(x[q], olo), ohi);
                Vec<T> o;
                o.pack(x);
                o.store(out, i);
                if (out2) o.store(out2, i);
            }
        }
    }
}

template <typename T, int V> static void ew_add_launch(const ValSrc& a, const ValSrc& b, int act, size_t n, int c, void* out, void* out2, cudaStream_t st) {
    size_t groups = n / V;
    LaunchScope ls(K_EW_ADD, (double)n * sizeof(T) * (1 + (b.p ? 1 : 0) + 1 + (out2 ? 1 : 0)), (double)n, st);
    if (V > 1) {
        const int vpr = c / V;
        size_t blocks = (groups + 4 * 256 - 1) / (4 * 256);
        const size_t cap = (size_t)sm_count() * 8;
        if (blocks > cap) blocks = cap;
        size_t threads = blocks * 256;
        if (threads < (size_t)vpr) {
            blocks = ((size_t)vpr + 255) / 256;
            threads = blocks * 256;
        }
        const size_t stride = threads / vpr * vpr;
        launch_pdl(ew_add_vec_kernel<T, V>, (unsigned)blocks, 256, 0, st, a, b, act, groups, vpr, stride, (T*)out, (T*)out2);
        return;
    }
    launch_pdl(ew_add_kernel<T, V>, (unsigned)((groups + 255) / 256), 256, 0, st, a, b, act, groups, c, (T*)out, (T*)out2);
}

void ew_add(int dtype, const ValSrc& a, const ValSrc& b, int act, size_t pixels, int c, void* out, void* out2, cudaStream_t st) {
    size_t n = pixels * c;
    if (dtype == 0) {
        if (c % 4 == 0) ew_add_launch<float, 4>(a, b, act, n, c, out, out2, st);
        else ew_add_launch<float, 1>(a, b, act, n, c, out, out2, st);
    } else {
        if (c % 8 == 0) ew_add_launch<__nv_bfloat16, 8>(a, b, act, n, c, out, out2, st);
        else ew_add_launch<__nv_bfloat16, 1>(a, b, act, n, c, out, out2, st);
    }
}

void ew_apply(int dtype, const ValSrc& a, size_t pixels, int c, void* out, cudaStream_t st) {
    ValSrc none{nullptr, nullptr, nullptr, 0};
    ew_add(dtype, a, none, ACT_NONE, pixels, c, out, nullptr, st);
}

template <typename T, int V> static void ew_flat_launch(int mode, const void* a, const void* b, size_t n, void* dst, cudaStream_t st) {
    size_t groups = n / V;
    LaunchScope ls(mode == 0 ? K_EW_MASK : K_EW_SUM, 3.0 * n * sizeof(T), (double)n, st);
    launch_pdl(ew_flat_kernel<T, V>, (unsigned)((groups + 255) / 256), 256, 0, st, mode, (const T*)a, (const T*)b, groups, (T*)dst);
}

static void ew_flat(int dtype, int mode, const void* a, const void* b, size_t n, void* dst, cudaStream_t st) {
    if (dtype == 0) {
        if (n % 4 == 0) ew_flat_launch<float, 4>(mode, a, b, n, dst, st);
        else ew_flat_launch<float, 1>(mode, a, b, n, dst, st);
    } else {
        if (n % 8 == 0) ew_flat_launch<__nv_bfloat16, 8>(mode, a, b, n, dst, st);
        else ew_flat_launch<__nv_bfloat16, 1>(mode, a, b, n, dst, st);
    }
}

void ew_relu_mask(int dtype, const void* d, const void* out_val, size_t n, void* dst, cudaStream_t st) { ew_flat(dtype, 0, d, out_val, n, dst, st); }
void ew_sum(int dtype, const void* a, const void* b, size_t n, void* dst, cudaStream_t st) { ew_flat(dtype, 1, a, b, n, dst, st); }

void ew_upsample2_grad(const GradSrc& d, int n, int hi, int wi, int ho, int wo, int c, void* up, cudaStream_t st) {
    const size_t groups = (size_t)n * hi * wi * (c / 8);
    LaunchScope ls(K_EW_SUM, 2.0 * ((double)n * ho * wo * c * ((d.act != ACT_NONE || d.k1) ? 2.0 : 1.0) + (double)n * hi * wi * c), 0.0, st);
    launch_pdl(ew_upsample2_kernel<__nv_bfloat16, 8>, (unsigned)((groups + 255) / 256), 256, 0, st, d, hi, wi, ho, wo, c, groups, (__nv_bfloat16*)up);
}

void ew_subsample2(const void* full, int n, int hi, int wi, int ho, int wo, int c, void* z, cudaStream_t st) {
    const size_t groups = (size_t)n * ho * wo * (c / 8);
    LaunchScope ls(K_EW_SUM, 4.0 * (double)n * ho * wo * c, 0.0, st);
    launch_pdl(ew_subsample2_kernel<__nv_bfloat16, 8>, (unsigned)((groups + 255) / 256), 256, 0, st, (const __nv_bfloat16*)full, hi, wi, ho, wo, c, groups,
               (__nv_bfloat16*)z);
}

void gap_fwd(int dtype, const ValSrc& x, int n, int hw, int c, void* out, cudaStream_t st) {
    int total = n * c;
    LaunchScope ls(K_GAP_FWD, ((double)total * hw + total) * esz(dtype), (double)total * hw, st);
    if (dtype == 0) launch_pdl(gap_fwd_kernel<float>, (total + 127) / 128, 128, 0, st, x, n, hw, c, (float*)out);
    else launch_pdl(gap_fwd_kernel<__nv_bfloat16>, (total + 127) / 128, 128, 0, st, x, n, hw, c, (__nv_bfloat16*)out);
}

void gap_bwd(int dtype, const void* da, int n, int hw, int c, const void* addend, void* dx, cudaStream_t st) {
    size_t total = (size_t)n * hw * c;
    unsigned blocks = (unsigned)((total + 255) / 256);
    LaunchScope ls(K_GAP_BWD, (double)total * esz(dtype) * (addend ? 2.0 : 1.0), (double)total, st);
    if (dtype == 0) launch_pdl(gap_bwd_kernel<float>, blocks, 256, 0, st, (const float*)da, n, hw, c, (const float*)addend, (float*)dx);
    else launch_pdl(gap_bwd_kernel<__nv_bfloat16>, blocks, 256, 0, st, (const __nv_bfloat16*)da, n, hw, c, (const __nv_bfloat16*)addend, (__nv_bfloat16*)dx);
}

void accumulate(float* G, const float* g, size_t n, cudaStream_t st) {
    if (!n) return;
    size_t n4 = n / 4, threads = n4 + (n - n4 * 4);
    LaunchScope ls(K_ACCUMULATE, 12.0 * n, (double)n, st);
    launch_pdl(accumulate_kernel, (unsigned)((threads + 255) / 256), 256, 0, st, G, g, n4, n);
}

void sgd_step(float* w, float* v, float* G, size_t n, float inv_m, float lr, float mu, cudaStream_t st) {
    if (!n) return;
    size_t n4 = n / 4, threads = n4 + (n - n4 * 4);
    LaunchScope ls(K_SGD_STEP, 24.0 * n, 5.0 * n, st);
    launch_pdl(sgd_step_kernel, (unsigned)((threads + 255) / 256), 256, 0, st, w, v, G, n4, n, inv_m, lr, mu);
}

void refresh_derived(const float* w, const int32_t* perm, float* derived, __nv_bfloat16* wb, __nv_bfloat16* wtb, size_t n, cudaStream_t st) {
    if (!n) return;
    LaunchScope ls(K_REFRESH, (wb ? 20.0 : 12.0) * n, 0.0, st);
    launch_pdl(refresh_kernel, (unsigned)((n + 255) / 256), 256, 0, st, w, perm, derived, wb, wtb, n);
}

// The MSE head's kernel for both entry points: the vector form where the three tensors are 16-byte aligned, else the scalar form.
static void launch_mse(int dtype, const void* y, const void* t, size_t n, void* dy, float* loss, float* scratch, unsigned* ticket, cudaStream_t st) {
    const bool vec = ((reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(t) | reinterpret_cast<uintptr_t>(dy)) & 15) == 0;
    const size_t per_block = vec ? (size_t)256 * 2 * (dtype == 0 ? 4 : 8) : (size_t)256 * 8;
    size_t want = (n + per_block - 1) / per_block;
    int blocks = (int)(want < 1 ? 1 : (want > LOSS_MAX_BLOCKS ? LOSS_MAX_BLOCKS : want));
    LaunchScope ls(K_LOSS_MSE, 3.0 * n * esz(dtype), 4.0 * n, st);
    if (dtype == 0) {
        if (vec) launch_pdl(mse_vec_kernel<float>, blocks, 256, 0, st, (const float*)y, (const float*)t, n, (float*)dy, loss, scratch, ticket);
        else launch_pdl(mse_kernel<float>, blocks, 256, 0, st, (const float*)y, (const float*)t, n, (float*)dy, loss, scratch, ticket);
    } else {
        if (vec) launch_pdl(mse_vec_kernel<__nv_bfloat16>, blocks, 256, 0, st, (const __nv_bfloat16*)y, (const __nv_bfloat16*)t, n, (__nv_bfloat16*)dy, loss, scratch, ticket);
        else launch_pdl(mse_kernel<__nv_bfloat16>, blocks, 256, 0, st, (const __nv_bfloat16*)y, (const __nv_bfloat16*)t, n, (__nv_bfloat16*)dy, loss, scratch, ticket);
    }
}

void loss_mse(int dtype, const void* y, const void* t, size_t n, void* dy, float* loss, float* scratch, cudaStream_t st) {
    launch_mse(dtype, y, t, n, dy, loss, scratch, reinterpret_cast<unsigned*>(scratch + 65536), st);
}

void loss_xent(int dtype, const void* logits, const int32_t* labels, int rows, int classes, void* dlogits, float* loss, float* scratch,
               cudaStream_t st) {
    unsigned* ticket = reinterpret_cast<unsigned*>(scratch + 65536);
    LaunchScope ls(K_LOSS_XENT, 2.0 * rows * classes * esz(dtype), 6.0 * rows * classes, st);
    if (dtype == 0) launch_pdl(xent_kernel<float>, rows, 256, 0, st, (const float*)logits, labels, rows, classes, (float*)dlogits, loss, scratch, ticket);
    else launch_pdl(xent_kernel<__nv_bfloat16>, rows, 256, 0, st, (const __nv_bfloat16*)logits, labels, rows, classes, (__nv_bfloat16*)dlogits, loss, scratch, ticket);
}

}  // namespace ast

// =================================================================== allocation-free MSE head
namespace ast {
namespace {
constexpr size_t NOALLOC_MAX_ELEMS = (size_t)1 << 26;
// Scratch of the allocation-free MSE head: one partial sum per block, then the ticket word.
// Lives in every GPU context that loads the library, until the process exits.
static __device__ __align__(256) float g_noalloc_scratch[LOSS_MAX_BLOCKS + 64];
// Device address of the array per device ordinal; the array's name is only a host-side handle,
// the address a kernel can use comes from cudaGetSymbolAddress with that device current.
float* g_noalloc_ptr[64] = {};
}  // namespace
}  // namespace ast

extern "C" int asteroid_loss_mse_noalloc(const void* y, const void* target, size_t n, int dtype, void* dy, float* loss, void* stream) {
    using namespace ast;
    if (!y || !target || !dy || !loss || n == 0) return report_error(-1, "asteroid_loss_mse_noalloc: null or empty argument");
    if (dtype != 0 && dtype != 1) return report_error(-1, "asteroid_loss_mse_noalloc: bad dtype");
    if (n > NOALLOC_MAX_ELEMS)
        return report_error(-1, "asteroid_loss_mse_noalloc: n exceeds the 67108864-element limit of the allocation-free variant; use asteroid_loss_mse");
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return report_error(-5, "asteroid_loss_mse_noalloc: cudaGetDevice failed");
    if (dev < 0 || dev >= 64) return report_error(-1, "asteroid_loss_mse_noalloc: device ordinals of 64 and above are not supported");
    // two host threads making the first call on a device at once both look up and store the same address: harmless
    if (!g_noalloc_ptr[dev]) {
        float* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) return report_error(-5, "asteroid_loss_mse_noalloc: cudaGetSymbolAddress failed");
        g_noalloc_ptr[dev] = p;
    }
    float* scratch = g_noalloc_ptr[dev];
    unsigned* ticket = reinterpret_cast<unsigned*>(scratch + LOSS_MAX_BLOCKS);
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the ticket must start at zero
    if (cudaMemsetAsync(ticket, 0, sizeof(unsigned), st) != cudaSuccess) return report_error(-5, "asteroid_loss_mse_noalloc: cudaMemsetAsync failed");
    launch_mse(dtype, y, target, n, dy, loss, scratch, ticket, st);
    if (cudaGetLastError() != cudaSuccess) return report_error(-5, "asteroid_loss_mse_noalloc: kernel launch failed");
    return 0;
}
