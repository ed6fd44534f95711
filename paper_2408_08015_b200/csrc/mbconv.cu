// Pieces of the EfficientNet MBConv block that the MobileNetV2 / ResNet kernels do not cover: the SiLU activation as a
// materialising elementwise unit (forward and backward), the squeeze-excite layer (per-sample channel means, two tiny
// fully connected layers, channel gate; forward and backward), and a depthwise convolution of any odd kernel size up to
// 7 (the 5x5 layers of the network).  All are bandwidth-bound passes over [pixels][channels] tensors with the producer's
// BatchNorm / activation applied while loading; reductions are two-stage and in fixed order (no float atomics).
#include "kernels.h"

namespace ast {
namespace {

// Per-thread register coefficients of one vector of V channels: value = clamp(z*scale+shift, lo, hi).
template <int V> struct ChanVal {
    float sc[V], sh[V], lo, hi;
    __device__ __forceinline__ void init(const ValSrc& s, int c0) {
#pragma unroll
        for (int q = 0; q < V; ++q) {
            sc[q] = s.scale ? __ldg(s.scale + c0 + q) : 1.f;
            sh[q] = s.scale ? __ldg(s.shift + c0 + q) : 0.f;
        }
        lo = s.act == ACT_NONE ? -INFINITY : 0.f;
        hi = s.act == ACT_RELU6 ? 6.f : INFINITY;
    }
    __device__ __forceinline__ void apply(float* f) const {
#pragma unroll
        for (int q = 0; q < V; ++q) f[q] = fminf(fmaxf(fmaf(f[q], sc[q], sh[q]), lo), hi);
    }
};
// dz = k1*dy*[lo < pre < hi] + k2 + k3*z, pre = z*scale+shift
template <int V> struct ChanGrad {
    float sc[V], sh[V], k1[V], k2[V], k3[V], lo, hi;
    bool need_z;
    __device__ __forceinline__ void init(const GradSrc& s, int c0) {
#pragma unroll
        for (int q = 0; q < V; ++q) {
            sc[q] = s.scale ? __ldg(s.scale + c0 + q) : 1.f;
            sh[q] = s.scale ? __ldg(s.shift + c0 + q) : 0.f;
            k1[q] = s.k1 ? __ldg(s.k1 + c0 + q) : 1.f;
            k2[q] = s.k1 ? __ldg(s.k2 + c0 + q) : 0.f;
            k3[q] = s.k1 ? __ldg(s.k3 + c0 + q) : 0.f;
        }
        lo = s.act == ACT_NONE ? -INFINITY : 0.f;
        hi = s.act == ACT_RELU6 ? 6.f : INFINITY;
        need_z = grad_needs_z(s);
    }
    __device__ __forceinline__ void apply(float* d, const float* z) const {
        if (!need_z) return;
#pragma unroll
        for (int q = 0; q < V; ++q) {
            const float pre = fmaf(z[q], sc[q], sh[q]);
            const float m = (pre > lo && pre < hi) ? d[q] : 0.f;
            d[q] = fmaf(k1[q], m, fmaf(k3[q], z[q], k2[q]));
        }
    }
};

__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + __expf(-x)); }

// Threads beyond `stride` (the thread count cut to a multiple of the vectors per pixel) idle, so that a thread striding by
// `stride` vectors always lands on the same channels.
struct VecGrid {
    unsigned blocks;
    size_t stride;
};
VecGrid vec_grid(size_t groups, int vpr, int per_thread) {
    size_t blocks = (groups + (size_t)per_thread * 256 - 1) / ((size_t)per_thread * 256);
    const size_t cap = (size_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    size_t threads = blocks * 256;
    if (threads < (size_t)vpr) {
        blocks = ((size_t)vpr + 255) / 256;
        threads = blocks * 256;
    }
    return VecGrid{(unsigned)blocks, threads / vpr * vpr};
}

// ------------------------------------------------------------------------------------------ SiLU
// forward: out = silu(value(x)); backward: dx = dy * silu'(value(x)) (+ addend), value(x) recomputed from the raw tensor
template <typename T, int V, bool BWD>
__global__ void __launch_bounds__(256) silu_kernel(ValSrc x, const T* __restrict__ dy, const T* addend, size_t groups, int vpr, size_t stride,
                                                   T* __restrict__ out, T* __restrict__ out2) {
    pdl_wait();
    pdl_launch();
    const size_t id = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= stride) return;
    ChanVal<V> cv;
    cv.init(x, (int)(id % (size_t)vpr) * V);
    for (size_t i = id; i < groups; i += stride) {
        float p[V], d[V], a[V];
        ld_raw_w<T, V>(x.p, i * V, p);
        cv.apply(p);
        if (BWD) {
            ld_raw_w<T, V>(dy, i * V, d);
            if (addend) ld_raw_w<T, V>(addend, i * V, a);
#pragma unroll
            for (int q = 0; q < V; ++q) {
                const float sg = sigmoidf_(p[q]);
                p[q] = d[q] * sg * fmaf(p[q], 1.f - sg, 1.f) + (addend ? a[q] : 0.f);
            }
        } else {
#pragma unroll
            for (int q = 0; q < V; ++q) p[q] = p[q] * sigmoidf_(p[q]);
        }
        st_raw_w<T, V>(out, i * V, p);
        if (out2) st_raw_w<T, V>(out2, i * V, p);
    }
}

// ------------------------------------------------------------------------------------------ squeeze-excite
// partial[n][rg][c] = sum over the pixels rg, rg+RG, ... of sample n of a[p][c] (MODE 0) or of d[p][c]*a[p][c] (MODE 1);
// a = value(x).  One block per (sample, group of 32*V channels), RG = 8 pixel classes; the classes are added in fixed order.
template <typename T, int V, int MODE>
__global__ void __launch_bounds__(256) se_reduce_kernel(ValSrc x, const T* __restrict__ d, int hw, int c, float scale, float* __restrict__ out) {
    pdl_wait();
    pdl_launch();
    __shared__ float sh[8][32 * V];
    const int n = blockIdx.y, lane = threadIdx.x & 31, rg = threadIdx.x >> 5;
    const int c0 = (blockIdx.x * 32 + lane) * V;
    float acc[V];
#pragma unroll
    for (int q = 0; q < V; ++q) acc[q] = 0.f;
    if (c0 < c) {
        ChanVal<V> cv;
        cv.init(x, c0);
        for (int p = rg; p < hw; p += 8) {
            const size_t e = ((size_t)n * hw + p) * c + c0;
            float a[V], g[V];
            ld_raw_w<T, V>(x.p, e, a);
            cv.apply(a);
            if (MODE == 1) {
                ld_raw_w<T, V>(d, e, g);
#pragma unroll
                for (int q = 0; q < V; ++q) acc[q] = fmaf(g[q], a[q], acc[q]);
            } else {
#pragma unroll
                for (int q = 0; q < V; ++q) acc[q] += a[q];
            }
        }
    }
#pragma unroll
    for (int q = 0; q < V; ++q) sh[rg][lane * V + q] = acc[q];
    __syncthreads();
    if (rg == 0 && c0 < c) {
#pragma unroll
        for (int q = 0; q < V; ++q) {
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) s += sh[k][lane * V + q];
            out[(size_t)n * c + c0 + q] = s * scale;
        }
    }
}

// One block per sample: p1 = w1 s + b1, h = silu(p1), g = sigmoid(w2 h + b2).  Keeps p1 and g for the backward pass.
__global__ void __launch_bounds__(256) se_fc_fwd_kernel(const float* __restrict__ s, const float* __restrict__ w1, const float* __restrict__ b1,
                                                        const float* __restrict__ w2, const float* __restrict__ b2, int c, int k,
                                                        float* __restrict__ p1, float* __restrict__ g) {
    pdl_wait();
    pdl_launch();
    extern __shared__ float hs[];              // h[k]
    const int n = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float* sn = s + (size_t)n * c;
    for (int j = warp; j < k; j += 8) {
        float acc = 0.f;
        for (int i = lane; i < c; i += 32) acc = fmaf(__ldg(w1 + (size_t)j * c + i), sn[i], acc);
        acc = warp_sum(acc) + __ldg(b1 + j);
        if (lane == 0) {
            p1[(size_t)n * k + j] = acc;
            hs[j] = acc * sigmoidf_(acc);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < c; i += 256) {
        float acc = __ldg(b2 + i);
        for (int j = 0; j < k; ++j) acc = fmaf(__ldg(w2 + (size_t)i * k + j), hs[j], acc);
        g[(size_t)n * c + i] = sigmoidf_(acc);
    }
}

// One block per sample: dp2 = dg g (1-g); dh = w2^T dp2; dp1 = dh silu'(p1); ds = w1^T dp1 / hw.
__global__ void __launch_bounds__(256) se_fc_bwd_kernel(const float* __restrict__ dg, const float* __restrict__ g, const float* __restrict__ p1,
                                                        const float* __restrict__ w1, const float* __restrict__ w2, int c, int k, float inv_hw,
                                                        float* __restrict__ dp2, float* __restrict__ dp1, float* __restrict__ ds) {
    pdl_wait();
    pdl_launch();
    extern __shared__ float sm[];              // dp2[c], dp1[k]
    float* sdp2 = sm;
    float* sdp1 = sm + c;
    const int n = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < c; i += 256) {
        const float gg = g[(size_t)n * c + i];
        const float v = dg[(size_t)n * c + i] * gg * (1.f - gg);
        sdp2[i] = v;
        dp2[(size_t)n * c + i] = v;
    }
    __syncthreads();
    for (int j = warp; j < k; j += 8) {
        float acc = 0.f;
        for (int i = lane; i < c; i += 32) acc = fmaf(__ldg(w2 + (size_t)i * k + j), sdp2[i], acc);
        acc = warp_sum(acc);
        if (lane == 0) {
            const float p = p1[(size_t)n * k + j], sg = sigmoidf_(p);
            const float v = acc * sg * fmaf(p, 1.f - sg, 1.f);
            sdp1[j] = v;
            dp1[(size_t)n * k + j] = v;
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < c; i += 256) {
        float acc = 0.f;
        for (int j = 0; j < k; ++j) acc = fmaf(__ldg(w1 + (size_t)j * c + i), sdp1[j], acc);
        ds[(size_t)n * c + i] = acc * inv_hw;       // the squeeze is a mean: every position of the sample receives ds / hw
    }
}

// Parameter gradients, one thread per parameter, samples added in index order:
// gw1[j][i] = sum_n dp1[n][j] s[n][i]; gb1[j] = sum_n dp1[n][j]; gw2[i][j] = sum_n dp2[n][i] h[n][j]; gb2[i] = sum_n dp2[n][i]
__global__ void __launch_bounds__(256) se_param_grad_kernel(const float* __restrict__ s, const float* __restrict__ p1, const float* __restrict__ dp1,
                                                            const float* __restrict__ dp2, int nb, int c, int k, float* __restrict__ gw1,
                                                            float* __restrict__ gb1, float* __restrict__ gw2, float* __restrict__ gb2) {
    pdl_wait();
    pdl_launch();
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int n_w = k * c;
    if (t < n_w) {                              // w1[j][i]
        const int j = t / c, i = t - j * c;
        float acc = 0.f;
        for (int n = 0; n < nb; ++n) acc = fmaf(dp1[(size_t)n * k + j], s[(size_t)n * c + i], acc);
        gw1[t] = acc;
    } else if (t < 2 * n_w) {                   // w2[i][j]
        const int u = t - n_w, i = u / k, j = u - i * k;
        float acc = 0.f;
        for (int n = 0; n < nb; ++n) {
            const float p = p1[(size_t)n * k + j];
            acc = fmaf(dp2[(size_t)n * c + i], p * sigmoidf_(p), acc);
        }
        gw2[u] = acc;
    } else if (t < 2 * n_w + k) {
        const int j = t - 2 * n_w;
        float acc = 0.f;
        for (int n = 0; n < nb; ++n) acc += dp1[(size_t)n * k + j];
        gb1[j] = acc;
    } else if (t < 2 * n_w + k + c) {
        const int i = t - 2 * n_w - k;
        float acc = 0.f;
        for (int n = 0; n < nb; ++n) acc += dp2[(size_t)n * c + i];
        gb2[i] = acc;
    }
}

// MODE 0: out = value(x) * gate[n][c];  MODE 1: out = d * gate[n][c] + ds[n][c] (+ addend), ds being the per-position share of the squeeze's gradient
template <typename T, int V, int MODE>
__global__ void __launch_bounds__(256) se_scale_kernel(ValSrc x, const T* __restrict__ d, const float* __restrict__ gate, const float* __restrict__ ds,
                                                       const T* addend, size_t groups, int vpr, int hw, size_t stride, T* __restrict__ out,
                                                       T* __restrict__ out2) {
    pdl_wait();
    pdl_launch();
    const size_t id = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= stride) return;
    const int c0 = (int)(id % (size_t)vpr) * V, c = vpr * V;
    ChanVal<V> cv;
    if (MODE == 0) cv.init(x, c0);
    for (size_t i = id; i < groups; i += stride) {
        const size_t n = (i / (size_t)vpr) / (size_t)hw;
        float v[V], a[V];
        if (MODE == 0) {
            ld_raw_w<T, V>(x.p, i * V, v);
            cv.apply(v);
#pragma unroll
            for (int q = 0; q < V; ++q) v[q] *= gate[n * c + c0 + q];
        } else {
            ld_raw_w<T, V>(d, i * V, v);
            if (addend) ld_raw_w<T, V>(addend, i * V, a);
#pragma unroll
            for (int q = 0; q < V; ++q) v[q] = fmaf(v[q], gate[n * c + c0 + q], ds[n * c + c0 + q]) + (addend ? a[q] : 0.f);
        }
        st_raw_w<T, V>(out, i * V, v);
        if (out2) st_raw_w<T, V>(out2, i * V, v);
    }
}

// ------------------------------------------------------------------------------------------ depthwise k x k
// weights tap-major wkc[t][c], t = r*k + s.  A thread owns V channels and walks output (or input) positions.
template <typename T, int V>
__global__ void __launch_bounds__(256) dwk_fwd_kernel(ConvGeom g, ValSrc x, const float* __restrict__ wkc, size_t groups, int vpr, size_t stride,
                                                      T* __restrict__ z) {
    pdl_wait();
    pdl_launch();
    const size_t id = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= stride) return;
    const int c0 = (int)(id % (size_t)vpr) * V, c = g.ci;
    ChanVal<V> cv;
    cv.init(x, c0);
    for (size_t i = id; i < groups; i += stride) {
        size_t pix = i / (size_t)vpr;
        const int wo = (int)(pix % g.wo);
        pix /= g.wo;
        const int ho = (int)(pix % g.ho), n = (int)(pix / g.ho);
        float acc[V];
#pragma unroll
        for (int q = 0; q < V; ++q) acc[q] = 0.f;
        for (int r = 0; r < g.k; ++r) {
            const int hi = ho * g.stride - g.pad + r;
            if (hi < 0 || hi >= g.hi) continue;
            for (int s = 0; s < g.k; ++s) {
                const int wi = wo * g.stride - g.pad + s;
                if (wi < 0 || wi >= g.wi) continue;
                float a[V];
                ld_raw_w<T, V>(x.p, (((size_t)n * g.hi + hi) * g.wi + wi) * c + c0, a);
                cv.apply(a);
                const float* wt = wkc + (size_t)(r * g.k + s) * c + c0;
#pragma unroll
                for (int q = 0; q < V; ++q) acc[q] = fmaf(a[q], __ldg(wt + q), acc[q]);
            }
        }
        st_raw_w<T, V>(z, i * V, acc);
    }
}

// dx[n,hi,wi,c] = sum_{r,s} dz[n,(hi+pad-r)/st,(wi+pad-s)/st,c] w[c][r][s] over the taps where the divisions are exact
template <typename T, int V>
__global__ void __launch_bounds__(256) dwk_bwd_data_kernel(ConvGeom g, GradSrc dz, const float* __restrict__ wkc, const T* addend, size_t groups, int vpr,
                                                           size_t stride, T* __restrict__ dx) {
    pdl_wait();
    pdl_launch();
    const size_t id = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= stride) return;
    const int c0 = (int)(id % (size_t)vpr) * V, c = g.ci;
    ChanGrad<V> cg;
    cg.init(dz, c0);
    for (size_t i = id; i < groups; i += stride) {
        size_t pix = i / (size_t)vpr;
        const int wi = (int)(pix % g.wi);
        pix /= g.wi;
        const int hi = (int)(pix % g.hi), n = (int)(pix / g.hi);
        float acc[V];
#pragma unroll
        for (int q = 0; q < V; ++q) acc[q] = 0.f;
        for (int r = 0; r < g.k; ++r) {
            const int hn = hi + g.pad - r;
            if (hn < 0 || hn % g.stride) continue;
            const int ho = hn / g.stride;
            if (ho >= g.ho) continue;
            for (int s = 0; s < g.k; ++s) {
                const int wn = wi + g.pad - s;
                if (wn < 0 || wn % g.stride) continue;
                const int wo = wn / g.stride;
                if (wo >= g.wo) continue;
                const size_t e = (((size_t)n * g.ho + ho) * g.wo + wo) * c + c0;
                float d[V], zz[V];
                ld_raw_w<T, V>(dz.dy, e, d);
                if (cg.need_z) ld_raw_w<T, V>(dz.z, e, zz);
                cg.apply(d, zz);
                const float* wt = wkc + (size_t)(r * g.k + s) * c + c0;
#pragma unroll
                for (int q = 0; q < V; ++q) acc[q] = fmaf(d[q], __ldg(wt + q), acc[q]);
            }
        }
        if (addend) {
            float a[V];
            ld_raw_w<T, V>(addend, i * V, a);
#pragma unroll
            for (int q = 0; q < V; ++q) acc[q] += a[q];
        }
        st_raw_w<T, V>(dx, i * V, acc);
    }
}

// partial[block][t][c] = sum over the block's output positions of dz[p][c] * x[p's tap t][c]; blockIdx.x = channel group of
// 32*V channels, blockIdx.y = position range; thread (lane, pg) walks positions pg, pg+4, ... of the range.  One tap
// row (k taps) per pass keeps the accumulators in registers.
template <typename T, int V>
__global__ void __launch_bounds__(128) dwk_bwd_weight_kernel(ConvGeom g, GradSrc dz, ValSrc x, size_t pos_per_block, float* __restrict__ partial) {
    pdl_wait();
    pdl_launch();
    __shared__ float sh[4][32 * V];
    const int lane = threadIdx.x & 31, pg = threadIdx.x >> 5;
    const int c = g.ci, c0 = (blockIdx.x * 32 + lane) * V;
    const bool live = c0 < c;
    const size_t total = (size_t)g.n * g.ho * g.wo;
    const size_t pbeg = (size_t)blockIdx.y * pos_per_block, pend = min(total, pbeg + pos_per_block);
    ChanGrad<V> cg;
    ChanVal<V> cv;
    cg.init(dz, live ? c0 : 0);
    cv.init(x, live ? c0 : 0);
    for (int r = 0; r < g.k; ++r)
        for (int s = 0; s < g.k; ++s) {
            float acc[V];
#pragma unroll
            for (int q = 0; q < V; ++q) acc[q] = 0.f;
            if (live)
                for (size_t p = pbeg + pg; p < pend; p += 4) {
                    const int wo = (int)(p % g.wo);
                    const size_t t2 = p / g.wo;
                    const int ho = (int)(t2 % g.ho), n = (int)(t2 / g.ho);
                    const int hi = ho * g.stride - g.pad + r, wi = wo * g.stride - g.pad + s;
                    if (hi < 0 || hi >= g.hi || wi < 0 || wi >= g.wi) continue;
                    float d[V], zz[V], a[V];
                    ld_raw_w<T, V>(dz.dy, p * c + c0, d);
                    if (cg.need_z) ld_raw_w<T, V>(dz.z, p * c + c0, zz);
                    cg.apply(d, zz);
                    ld_raw_w<T, V>(x.p, (((size_t)n * g.hi + hi) * g.wi + wi) * c + c0, a);
                    cv.apply(a);
#pragma unroll
                    for (int q = 0; q < V; ++q) acc[q] = fmaf(d[q], a[q], acc[q]);
                }
#pragma unroll
            for (int q = 0; q < V; ++q) sh[pg][lane * V + q] = acc[q];
            __syncthreads();
            if (pg == 0 && live) {
#pragma unroll
                for (int q = 0; q < V; ++q)
                    partial[((size_t)blockIdx.y * g.k * g.k + (r * g.k + s)) * c + c0 + q] = sh[0][lane * V + q] + sh[1][lane * V + q] + sh[2][lane * V + q] + sh[3][lane * V + q];
            }
            __syncthreads();
        }
}

// gw[c][t] = sum over blocks (index order) of partial[b][t][c]
__global__ void __launch_bounds__(256) dwk_weight_finish_kernel(const float* __restrict__ partial, int blocks, int taps, int c, float* __restrict__ gw) {
    pdl_wait();
    pdl_launch();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= taps * c) return;
    const int t = i / c, ch = i - t * c;
    float s = 0.f;
    for (int b = 0; b < blocks; ++b) s += partial[((size_t)b * taps + t) * c + ch];
    gw[(size_t)ch * taps + t] = s;
}

double esz_(int dtype) { return dtype == 0 ? 4.0 : 2.0; }

}  // namespace

// runs the statement block with T (storage type) and V (channels per vector: 16 bytes where the channel count allows, else 1)
#define DISPATCH_TV(dtype, c, ...)                                                                \
    do {                                                                                          \
        if ((dtype) == 0) {                                                                       \
            if ((c) % 4 == 0) { using T = float; constexpr int V = 4; __VA_ARGS__ }               \
            else { using T = float; constexpr int V = 1; __VA_ARGS__ }                            \
        } else {                                                                                  \
            if ((c) % 8 == 0) { using T = __nv_bfloat16; constexpr int V = 8; __VA_ARGS__ }       \
            else { using T = __nv_bfloat16; constexpr int V = 1; __VA_ARGS__ }                    \
        }                                                                                         \
    } while (0)

void silu_fwd(int dtype, const ValSrc& x, size_t pixels, int c, void* out, void* out2, cudaStream_t st) {
    const size_t n = pixels * c;
    LaunchScope ls(K_SILU, (double)n * esz_(dtype) * (2 + (out2 ? 1 : 0)), 4.0 * n, st);
    DISPATCH_TV(dtype, c, {
        const VecGrid vg = vec_grid(n / V, c / V, 4);
        launch_pdl(silu_kernel<T, V, false>, vg.blocks, 256, 0, st, x, (const T*)nullptr, (const T*)nullptr, n / V, c / V, vg.stride, (T*)out, (T*)out2);
    });
}

void silu_bwd(int dtype, const void* dy, const ValSrc& x, const void* addend, size_t pixels, int c, void* dx, cudaStream_t st) {
    const size_t n = pixels * c;
    LaunchScope ls(K_SILU, (double)n * esz_(dtype) * (3 + (addend ? 1 : 0)), 8.0 * n, st);
    DISPATCH_TV(dtype, c, {
        const VecGrid vg = vec_grid(n / V, c / V, 4);
        launch_pdl(silu_kernel<T, V, true>, vg.blocks, 256, 0, st, x, (const T*)dy, (const T*)addend, n / V, c / V, vg.stride, (T*)dx, (T*)nullptr);
    });
}

void se_forward(int dtype, const ValSrc& x, int n, int hw, int c, int k, const float* w1, const float* b1, const float* w2, const float* b2,
                float* s, float* p1, float* gate, void* out, void* out2, cudaStream_t st) {
    const size_t elems = (size_t)n * hw * c;
    {
        LaunchScope ls(K_SE, (double)elems * esz_(dtype), (double)elems, st);
        DISPATCH_TV(dtype, c, { launch_pdl(se_reduce_kernel<T, V, 0>, dim3((c / V + 31) / 32, n), 256, 0, st, x, (const T*)nullptr, hw, c, 1.f / (float)hw, s); });
    }
    {
        LaunchScope ls(K_SE, 4.0 * (2.0 * k * c + (double)n * (2 * c + k)), 4.0 * n * k * c, st);
        launch_pdl(se_fc_fwd_kernel, n, 256, (size_t)k * sizeof(float), st, (const float*)s, w1, b1, w2, b2, c, k, p1, gate);
    }
    LaunchScope ls(K_SE, (double)elems * esz_(dtype) * (2 + (out2 ? 1 : 0)), (double)elems, st);
    DISPATCH_TV(dtype, c, {
        const VecGrid vg = vec_grid(elems / V, c / V, 4);
        launch_pdl(se_scale_kernel<T, V, 0>, vg.blocks, 256, 0, st, x, (const T*)nullptr, (const float*)gate, (const float*)nullptr, (const T*)nullptr, elems / V, c / V, hw,
                   vg.stride, (T*)out, (T*)out2);
    });
}

void se_backward(int dtype, const void* dout, const ValSrc& x, int n, int hw, int c, int k, const float* w1, const float* w2, const float* s,
                 const float* p1, const float* gate, float* work, const void* addend, void* dx, float* gw1, float* gb1, float* gw2, float* gb2,
                 cudaStream_t st) {
    const size_t elems = (size_t)n * hw * c;
    float* dg = work;                          // [n][c]
    float* dp2 = dg + (size_t)n * c;           // [n][c]
    float* ds = dp2 + (size_t)n * c;           // [n][c]
    float* dp1 = ds + (size_t)n * c;           // [n][k]
    {
        LaunchScope ls(K_SE, 2.0 * elems * esz_(dtype), 2.0 * elems, st);
        DISPATCH_TV(dtype, c, { launch_pdl(se_reduce_kernel<T, V, 1>, dim3((c / V + 31) / 32, n), 256, 0, st, x, (const T*)dout, hw, c, 1.f, dg); });
    }
    {
        LaunchScope ls(K_SE, 4.0 * (2.0 * k * c + (double)n * (4 * c + 2 * k)), 4.0 * n * k * c, st);
        launch_pdl(se_fc_bwd_kernel, n, 256, (size_t)(c + k) * sizeof(float), st, (const float*)dg, gate, p1, w1, w2, c, k, 1.f / (float)hw, dp2, dp1, ds);
    }
    {
        const int params = 2 * k * c + k + c;
        LaunchScope ls(K_SE, 4.0 * (params + (double)n * (2 * c + 2 * k)), 4.0 * n * k * c, st);
        launch_pdl(se_param_grad_kernel, (params + 255) / 256, 256, 0, st, s, p1, (const float*)dp1, (const float*)dp2, n, c, k, gw1, gb1, gw2, gb2);
    }
    if (!dx) return;                           // only the parameter gradients are wanted
    LaunchScope ls(K_SE, (double)elems * esz_(dtype) * (2 + (addend ? 1 : 0)), 2.0 * elems, st);
    DISPATCH_TV(dtype, c, {
        const VecGrid vg = vec_grid(elems / V, c / V, 4);
        launch_pdl(se_scale_kernel<T, V, 1>, vg.blocks, 256, 0, st, x, (const T*)dout, gate, (const float*)ds, (const T*)addend, elems / V, c / V, hw, vg.stride,
                   (T*)dx, (T*)nullptr);
    });
}

void dwk_fwd(int dtype, const ConvGeom& g, const ValSrc& x, const float* wkc, void* z, cudaStream_t st) {
    const size_t out_e = (size_t)g.n * g.ho * g.wo * g.ci, in_e = (size_t)g.n * g.hi * g.wi * g.ci;
    LaunchScope ls(K_DW_FWD, ((double)in_e + out_e) * esz_(dtype) + 4.0 * g.k * g.k * g.ci, 2.0 * g.k * g.k * out_e, st);
    DISPATCH_TV(dtype, g.ci, {
        const VecGrid vg = vec_grid(out_e / V, g.ci / V, 2);
        launch_pdl(dwk_fwd_kernel<T, V>, vg.blocks, 256, 0, st, g, x, wkc, out_e / V, g.ci / V, vg.stride, (T*)z);
    });
}

void dwk_bwd_data(int dtype, const ConvGeom& g, const GradSrc& dz, const float* wkc, const void* addend, void* dx, cudaStream_t st) {
    const size_t out_e = (size_t)g.n * g.ho * g.wo * g.ci, in_e = (size_t)g.n * g.hi * g.wi * g.ci;
    LaunchScope ls(K_DW_BWD_DATA, ((double)out_e * (grad_needs_z(dz) ? 2 : 1) + (double)in_e * (addend ? 2 : 1)) * esz_(dtype), 2.0 * g.k * g.k * out_e, st);
    DISPATCH_TV(dtype, g.ci, {
        const VecGrid vg = vec_grid(in_e / V, g.ci / V, 2);
        launch_pdl(dwk_bwd_data_kernel<T, V>, vg.blocks, 256, 0, st, g, dz, wkc, (const T*)addend, in_e / V, g.ci / V, vg.stride, (T*)dx);
    });
}

void dwk_bwd_weight(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw, cudaStream_t st) {
    const size_t positions = (size_t)g.n * g.ho * g.wo, out_e = positions * g.ci, in_e = (size_t)g.n * g.hi * g.wi * g.ci;
    const int taps = g.k * g.k;
    int by = 0;
    DISPATCH_TV(dtype, g.ci, {
        const int gx = (g.ci / V + 31) / 32;
        size_t want = ((size_t)4 * sm_count() + gx - 1) / gx;
        const size_t cap = scratch_floats / ((size_t)taps * g.ci);
        if (want > cap) want = cap;
        if (want > (positions + 15) / 16) want = (positions + 15) / 16;
        if (want < 1) want = 1;
        const size_t ppb = (positions + want - 1) / want;
        by = (int)((positions + ppb - 1) / ppb);
        LaunchScope ls(K_DW_BWD_WEIGHT, ((double)out_e * (grad_needs_z(dz) ? 2 : 1) + in_e) * esz_(dtype) + 4.0 * taps * g.ci * by, 2.0 * taps * out_e, st);
        launch_pdl(dwk_bwd_weight_kernel<T, V>, dim3(gx, by), 128, 0, st, g, dz, x, ppb, scratch);
    });
    LaunchScope ls(K_DW_BWD_WEIGHT_FINISH, 4.0 * taps * g.ci * (by + 1), (double)taps * g.ci * by, st);
    launch_pdl(dwk_weight_finish_kernel, (taps * g.ci + 255) / 256, 256, 0, st, (const float*)scratch, by, taps, g.ci, gw);
}

}  // namespace ast
