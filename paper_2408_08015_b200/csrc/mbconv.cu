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
// out[z][n][c] = sum over the pixels p = 8z+rg, 8z+rg+8Z, ... (rg = 0..7, Z = gridDim.z pixel splits) of sample n of a[p][c]
// (MODE 0) or of d[p][c]*a[p][c] (MODE 1); a = value(x).  One block per (group of 32*V channels, sample, split); the eight
// pixel classes of a block are added in fixed order, the splits by the consumer in index order.
template <typename T, int V, int MODE>
__global__ void __launch_bounds__(256) se_reduce_kernel(ValSrc x, const T* __restrict__ d, int hw, int c, float* __restrict__ out) {
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
        for (int p = blockIdx.z * 8 + rg; p < hw; p += 8 * gridDim.z) {
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
            out[((size_t)blockIdx.z * gridDim.y + n) * c + c0 + q] = s;
        }
    }
}

// One block per sample: s = (sum of the pixel-split partials) / hw, p1 = w1 s + b1, h = silu(p1), g = sigmoid(w2 h + b2).
// Keeps s, p1 and g for the backward pass.
__global__ void __launch_bounds__(256) se_fc_fwd_kernel(const float* __restrict__ part, int splits, float inv_hw, const float* __restrict__ w1,
                                                        const float* __restrict__ b1, const float* __restrict__ w2, const float* __restrict__ b2, int c, int k,
                                                        float* __restrict__ s, float* __restrict__ p1, float* __restrict__ g) {
    pdl_wait();
    pdl_launch();
    extern __shared__ float hs[];              // h[k], s[c]
    float* sn = hs + k;
    const int n = blockIdx.x, nb = gridDim.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < c; i += 256) {
        float a = 0.f;
        for (int z = 0; z < splits; ++z) a += part[((size_t)z * nb + n) * c + i];
        a *= inv_hw;
        sn[i] = a;
        s[(size_t)n * c + i] = a;
    }
    __syncthreads();
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

// One block per sample: dg = sum of the pixel-split partials; dp2 = dg g (1-g); dh = w2^T dp2; dp1 = dh silu'(p1); ds = w1^T dp1 / hw.
__global__ void __launch_bounds__(256) se_fc_bwd_kernel(const float* __restrict__ part, int splits, const float* __restrict__ g, const float* __restrict__ p1,
                                                        const float* __restrict__ w1, const float* __restrict__ w2, int c, int k, float inv_hw,
                                                        float* __restrict__ dp2, float* __restrict__ dp1, float* __restrict__ ds) {
    pdl_wait();
    pdl_launch();
    extern __shared__ float sm[];              // dp2[c], dp1[k]
    float* sdp2 = sm;
    float* sdp1 = sm + c;
    const int n = blockIdx.x, nb = gridDim.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < c; i += 256) {
        const float gg = g[(size_t)n * c + i];
        float dg = 0.f;                          // gradient of the gate: the pixel-split partials of sum dout*x, in index order
        for (int z = 0; z < splits; ++z) dg += part[((size_t)z * nb + n) * c + i];
        const float v = dg * gg * (1.f - gg);
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
// weights tap-major wkc[t][c], t = r*K + s, float32, read as 16-byte vectors through the read-only path.  A thread owns one
// vector of V = 4 channels and a horizontal strip of TW pixels: a row of the source tensor is loaded and
// transformed once per thread and feeds every (pixel, tap) pair of the strip it touches; kernel size and stride are
// compile-time, so the tap loops unroll completely and the per-row weights sit in registers.
// V channels starting at element e: 4 channels of either storage type (16 bytes of float, 8 of bfloat16), else the
// widths ld_raw_w / st_raw_w know
template <typename T, int V> __device__ __forceinline__ void ldv(const void* p, size_t e, float* out) {
    if constexpr (V == 4 && sizeof(T) == 2) {
        const uint2 r = *reinterpret_cast<const uint2*>(reinterpret_cast<const T*>(p) + e);
        out[0] = __uint_as_float(r.x << 16);
        out[1] = __uint_as_float(r.x & 0xffff0000u);
        out[2] = __uint_as_float(r.y << 16);
        out[3] = __uint_as_float(r.y & 0xffff0000u);
    } else {
        ld_raw_w<T, V>(p, e, out);
    }
}
template <typename T, int V> __device__ __forceinline__ void stv(void* p, size_t e, const float* in) {
    if constexpr (V == 4 && sizeof(T) == 2) {
        const __nv_bfloat162 a = __floats2bfloat162_rn(in[0], in[1]), b = __floats2bfloat162_rn(in[2], in[3]);
        uint2 r;
        r.x = *reinterpret_cast<const uint32_t*>(&a);
        r.y = *reinterpret_cast<const uint32_t*>(&b);
        *reinterpret_cast<uint2*>(reinterpret_cast<T*>(p) + e) = r;
    } else {
        st_raw_w<T, V>(p, e, in);
    }
}

template <int V> __device__ __forceinline__ void ld_w(const float* __restrict__ w, float* out) {
#pragma unroll
    for (int q = 0; q < V; q += 4) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(w + q));
        out[q] = t.x; out[q + 1] = t.y; out[q + 2] = t.z; out[q + 3] = t.w;
    }
}

struct StripIdx {
    int n, h, w0;
};
__device__ __forceinline__ StripIdx strip_of(size_t item, int vpr, int strips, int rows, int tw) {
    size_t sp = item / (size_t)vpr;
    StripIdx r;
    r.w0 = (int)(sp % strips) * tw;
    sp /= strips;
    r.h = (int)(sp % rows);
    r.n = (int)(sp / rows);
    return r;
}

// Forward (FLIP = false, SRC = ValSrc over x, S = stride) and stride-1 backward-data (FLIP = true, SRC = GradSrc over dz,
// S = 1: dx is the correlation of dz with the kernel turned by 180 degrees).  out[n][h][w0+t] for t < TW.
template <typename T, int V, int K, int S, int TW, bool FLIP, typename COEF, typename SRC>
__global__ void __launch_bounds__(256) dwk_strip_kernel(int hin, int win, int hout, int wout, int c, SRC src, const float* __restrict__ wkc, const T* addend,
                                                        size_t items, int strips, size_t stride, T* __restrict__ out) {
    pdl_wait();
    pdl_launch();
    constexpr int PAD = (K - 1) / 2, SPAN = (TW - 1) * S + K;
    const size_t id = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= stride) return;
    const int vpr = c / V, c0 = (int)(id % (size_t)vpr) * V;
    COEF cf;
    cf.init(src, c0);
    for (size_t i = id; i < items; i += stride) {
        const StripIdx q = strip_of(i, vpr, strips, hout, TW);
        float acc[TW][V];
#pragma unroll
        for (int t = 0; t < TW; ++t)
#pragma unroll
            for (int e = 0; e < V; ++e) acc[t][e] = 0.f;
#pragma unroll
        for (int r = 0; r < K; ++r) {
            const int hi = q.h * S - PAD + r;
            if ((unsigned)hi >= (unsigned)hin) continue;
            float wr[K][V];
#pragma unroll
            for (int s = 0; s < K; ++s) ld_w<V>(wkc + (size_t)(FLIP ? (K - 1 - r) * K + (K - 1 - s) : r * K + s) * c + c0, wr[s]);
            const size_t rowbase = ((size_t)q.n * hin + hi) * win;
#pragma unroll
            for (int j = 0; j < SPAN; ++j) {
                const int wi = q.w0 * S - PAD + j;
                float a[V];
                if ((unsigned)wi < (unsigned)win) cf.template load<T>(src, (rowbase + wi) * c + c0, a);
                else {
#pragma unroll
                    for (int e = 0; e < V; ++e) a[e] = 0.f;
                }
#pragma unroll
                for (int t = 0; t < TW; ++t) {
                    const int s = j - t * S;
                    if (s >= 0 && s < K) {
#pragma unroll
                        for (int e = 0; e < V; ++e) acc[t][e] = fmaf(a[e], wr[s][e], acc[t][e]);
                    }
                }
            }
        }
#pragma unroll
        for (int t = 0; t < TW; ++t) {
            if (q.w0 + t >= wout) break;
            const size_t e0 = (((size_t)q.n * hout + q.h) * wout + q.w0 + t) * c + c0;
            if (addend) {
                float ad[V];
                ldv<T, V>(addend, e0, ad);
#pragma unroll
                for (int e = 0; e < V; ++e) acc[t][e] += ad[e];
            }
            stv<T, V>(out, e0, acc[t]);
        }
    }
}

// loaders with the coefficients in registers
template <int V> struct ValCoef : ChanVal<V> {
    template <typename T> __device__ __forceinline__ void load(const ValSrc& s, size_t e, float* a) const {
        ldv<T, V>(s.p, e, a);
        this->apply(a);
    }
};
template <int V> struct GradCoef : ChanGrad<V> {
    template <typename T> __device__ __forceinline__ void load(const GradSrc& s, size_t e, float* d) const {
        float zz[V];
        ldv<T, V>(s.dy, e, d);
        if (this->need_z) ldv<T, V>(s.z, e, zz);
        this->apply(d, zz);
    }
};

// Stride-2 backward-data: dx[n][hi][wi0+t], t < TW (wi0 even, TW even), from the dz rows ho = (hi + PAD - r) / 2 of the taps r with
// hi + PAD - r even; along the row the column of dz that tap s of pixel t reads is wi0/2 + (t + PAD - s)/2 for t + PAD - s even:
// NCOL consecutive columns starting at wi0/2 + JLO, loaded once per row.
template <typename T, int V, int K, int TW>
__global__ void __launch_bounds__(256) dwk_bwd_data_s2_kernel(ConvGeom g, GradSrc dz, const float* __restrict__ wkc, const T* addend, size_t items, int strips,
                                                              size_t stride, T* __restrict__ dx) {
    pdl_wait();
    pdl_launch();
    constexpr int PAD = (K - 1) / 2;
    // (t + PAD - s) / 2 over even values of t + PAD - s, t in [0,TW), s in [0,K)
    constexpr int DLO = -((K - 1 - PAD) / 2), DHI = (TW - 1 + PAD) / 2, NCOL = DHI - DLO + 1;
    const size_t id = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= stride) return;
    const int c = g.ci, vpr = c / V, c0 = (int)(id % (size_t)vpr) * V;
    GradCoef<V> cf;
    cf.init(dz, c0);
    for (size_t i = id; i < items; i += stride) {
        const StripIdx q = strip_of(i, vpr, strips, g.hi, TW);
        float acc[TW][V];
#pragma unroll
        for (int t = 0; t < TW; ++t)
#pragma unroll
            for (int e = 0; e < V; ++e) acc[t][e] = 0.f;
        for (int r = (q.h + PAD) & 1; r < K; r += 2) {
            const int hn = q.h + PAD - r;
            if (hn < 0) break;
            const int ho = hn >> 1;
            if (ho >= g.ho) continue;
            float wr[K][V];
#pragma unroll
            for (int s = 0; s < K; ++s) ld_w<V>(wkc + (size_t)(r * K + s) * c + c0, wr[s]);
            const size_t rowbase = ((size_t)q.n * g.ho + ho) * g.wo;
#pragma unroll
            for (int j = 0; j < NCOL; ++j) {
                const int wo = (q.w0 >> 1) + DLO + j;
                float d[V];
                if ((unsigned)wo < (unsigned)g.wo) cf.template load<T>(dz, (rowbase + wo) * c + c0, d);
                else {
#pragma unroll
                    for (int e = 0; e < V; ++e) d[e] = 0.f;
                }
#pragma unroll
                for (int t = 0; t < TW; ++t)
#pragma unroll
                    for (int s = 0; s < K; ++s) {
                        if (((t + PAD - s) % 2 == 0) && ((t + PAD - s) / 2 == DLO + j)) {
#pragma unroll
                            for (int e = 0; e < V; ++e) acc[t][e] = fmaf(d[e], wr[s][e], acc[t][e]);
                        }
                    }
            }
        }
#pragma unroll
        for (int t = 0; t < TW; ++t) {
            if (q.w0 + t >= g.wi) break;
            const size_t e0 = (((size_t)q.n * g.hi + q.h) * g.wi + q.w0 + t) * c + c0;
            if (addend) {
                float ad[V];
                ldv<T, V>(addend, e0, ad);
#pragma unroll
                for (int e = 0; e < V; ++e) acc[t][e] += ad[e];
            }
            stv<T, V>(dx, e0, acc[t]);
        }
    }
}

// Weight gradient, one tap row r per pass: partial[block][r*K+s][c] = sum over the block's strips of dz[p] * x[p's tap (r,s)].
// blockIdx.x = group of 32 channel vectors (one per lane), blockIdx.y = range of strips (a strip = TW consecutive output
// pixels of one row); warp pg of the block takes strips pg, pg+4, ... of the range.
template <typename T, int V, int K, int S, int TW>
__global__ void __launch_bounds__(128) dwk_bwd_weight_kernel(ConvGeom g, GradSrc dz, ValSrc x, int strips, size_t strips_per_block, float* __restrict__ partial) {
    pdl_wait();
    pdl_launch();
    constexpr int PAD = (K - 1) / 2, SPAN = (TW - 1) * S + K;
    __shared__ float sh[4][32 * V];
    const int lane = threadIdx.x & 31, pg = threadIdx.x >> 5;
    const int c = g.ci, c0 = (blockIdx.x * 32 + lane) * V;
    const bool live = c0 < c;
    const size_t total = (size_t)g.n * g.ho * strips;
    const size_t sbeg = (size_t)blockIdx.y * strips_per_block, send = min(total, sbeg + strips_per_block);
    GradCoef<V> cg;
    ValCoef<V> cv;
    cg.init(dz, live ? c0 : 0);
    cv.init(x, live ? c0 : 0);
    for (int r = 0; r < K; ++r) {
        float acc[K][V];
#pragma unroll
        for (int s = 0; s < K; ++s)
#pragma unroll
            for (int e = 0; e < V; ++e) acc[s][e] = 0.f;
        if (live)
            for (size_t sp = sbeg + pg; sp < send; sp += 4) {
                const int w0 = (int)(sp % strips) * TW;
                const size_t t2 = sp / strips;
                const int ho = (int)(t2 % g.ho), n = (int)(t2 / g.ho);
                const int hi = ho * S - PAD + r;
                if ((unsigned)hi >= (unsigned)g.hi) continue;
                float d[TW][V];
#pragma unroll
                for (int t = 0; t < TW; ++t) {
                    if (w0 + t < g.wo) cg.template load<T>(dz, (((size_t)n * g.ho + ho) * g.wo + w0 + t) * c + c0, d[t]);
                    else {
#pragma unroll
                        for (int e = 0; e < V; ++e) d[t][e] = 0.f;
                    }
                }
                const size_t rowbase = ((size_t)n * g.hi + hi) * g.wi;
#pragma unroll
                for (int j = 0; j < SPAN; ++j) {
                    const int wi = w0 * S - PAD + j;
                    if ((unsigned)wi >= (unsigned)g.wi) continue;
                    float a[V];
                    cv.template load<T>(x, (rowbase + wi) * c + c0, a);
#pragma unroll
                    for (int t = 0; t < TW; ++t) {
                        const int s = j - t * S;
                        if (s >= 0 && s < K) {
#pragma unroll
                            for (int e = 0; e < V; ++e) acc[s][e] = fmaf(d[t][e], a[e], acc[s][e]);
                        }
                    }
                }
            }
#pragma unroll
        for (int s = 0; s < K; ++s) {
#pragma unroll
            for (int e = 0; e < V; ++e) sh[pg][lane * V + e] = acc[s][e];
            __syncthreads();
            if (pg == 0 && live) {
#pragma unroll
                for (int e = 0; e < V; ++e)
                    partial[((size_t)blockIdx.y * K * K + (r * K + s)) * c + c0 + e] = sh[0][lane * V + e] + sh[1][lane * V + e] + sh[2][lane * V + e] + sh[3][lane * V + e];
            }
            __syncthreads();
        }
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

// pixel splits of the squeeze reductions: enough blocks for two per SM, at least 32 pixels per block, within the scratch
static int se_splits(int gx, int n, int hw, int c, size_t scratch_floats) {
    int z = (2 * sm_count() + gx * n - 1) / (gx * n);
    if (z > hw / 32) z = hw / 32;
    const size_t cap = scratch_floats / ((size_t)n * c);
    if ((size_t)z > cap) z = (int)cap;
    return z < 1 ? 1 : z;
}

void se_forward(int dtype, const ValSrc& x, int n, int hw, int c, int k, const float* w1, const float* b1, const float* w2, const float* b2,
                float* s, float* p1, float* gate, float* scratch, size_t scratch_floats, void* out, void* out2, cudaStream_t st) {
    const size_t elems = (size_t)n * hw * c;
    int splits = 1;
    {
        LaunchScope ls(K_SE, (double)elems * esz_(dtype), (double)elems, st);
        DISPATCH_TV(dtype, c, {
            const int gx = (c / V + 31) / 32;
            splits = se_splits(gx, n, hw, c, scratch_floats);
            launch_pdl(se_reduce_kernel<T, V, 0>, dim3(gx, n, splits), 256, 0, st, x, (const T*)nullptr, hw, c, scratch);
        });
    }
    {
        LaunchScope ls(K_SE, 4.0 * (2.0 * k * c + (double)n * ((2 + splits) * c + k)), 4.0 * n * k * c, st);
        launch_pdl(se_fc_fwd_kernel, n, 256, (size_t)(k + c) * sizeof(float), st, (const float*)scratch, splits, 1.f / (float)hw, w1, b1, w2, b2, c, k, s, p1, gate);
    }
    LaunchScope ls(K_SE, (double)elems * esz_(dtype) * (2 + (out2 ? 1 : 0)), (double)elems, st);
    DISPATCH_TV(dtype, c, {
        const VecGrid vg = vec_grid(elems / V, c / V, 4);
        launch_pdl(se_scale_kernel<T, V, 0>, vg.blocks, 256, 0, st, x, (const T*)nullptr, (const float*)gate, (const float*)nullptr, (const T*)nullptr, elems / V, c / V, hw,
                   vg.stride, (T*)out, (T*)out2);
    });
}

void se_backward(int dtype, const void* dout, const ValSrc& x, int n, int hw, int c, int k, const float* w1, const float* w2, const float* s,
                 const float* p1, const float* gate, float* work, float* scratch, size_t scratch_floats, const void* addend, void* dx, float* gw1, float* gb1,
                 float* gw2, float* gb2, cudaStream_t st) {
    const size_t elems = (size_t)n * hw * c;
    float* dp2 = work;                         // [n][c]
    float* ds = dp2 + (size_t)n * c;           // [n][c]
    float* dp1 = ds + (size_t)n * c;           // [n][k]
    int splits = 1;
    {
        LaunchScope ls(K_SE, 2.0 * elems * esz_(dtype), 2.0 * elems, st);
        DISPATCH_TV(dtype, c, {
            const int gx = (c / V + 31) / 32;
            splits = se_splits(gx, n, hw, c, scratch_floats);
            launch_pdl(se_reduce_kernel<T, V, 1>, dim3(gx, n, splits), 256, 0, st, x, (const T*)dout, hw, c, scratch);
        });
    }
    {
        LaunchScope ls(K_SE, 4.0 * (2.0 * k * c + (double)n * ((3 + splits) * c + 2 * k)), 4.0 * n * k * c, st);
        launch_pdl(se_fc_bwd_kernel, n, 256, (size_t)(c + k) * sizeof(float), st, (const float*)scratch, splits, gate, p1, w1, w2, c, k, 1.f / (float)hw, dp2, dp1, ds);
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

// runs the statement block with T and V = 4 channels per thread (16 bytes of float, 8 of bfloat16: the wider bfloat16 vector
// costs twice the accumulator and coefficient registers and left one block per SM)
#define DISPATCH_T16(dtype, ...)                                                    \
    do {                                                                            \
        if ((dtype) == 0) { using T = float; constexpr int V = 4; __VA_ARGS__ }     \
        else { using T = __nv_bfloat16; constexpr int V = 4; __VA_ARGS__ }          \
    } while (0)
// ... and with the compile-time kernel size K in {5, 7}
#define DISPATCH_K(k, ...)                                  \
    do {                                                    \
        if ((k) == 5) { constexpr int K = 5; __VA_ARGS__ }  \
        else { constexpr int K = 7; __VA_ARGS__ }           \
    } while (0)

void dwk_fwd(int dtype, const ConvGeom& g, const ValSrc& x, const float* wkc, void* z, cudaStream_t st) {
    const size_t out_e = (size_t)g.n * g.ho * g.wo * g.ci, in_e = (size_t)g.n * g.hi * g.wi * g.ci;
    LaunchScope ls(K_DW_FWD, ((double)in_e + out_e) * esz_(dtype) + 4.0 * g.k * g.k * g.ci, 2.0 * g.k * g.k * out_e, st);
    DISPATCH_T16(dtype, DISPATCH_K(g.k, {
        constexpr int TW = 4;
        const int strips = (g.wo + TW - 1) / TW, vpr = g.ci / V;
        const size_t items = (size_t)g.n * g.ho * strips * vpr;
        const VecGrid vg = vec_grid(items, vpr, 1);
        if (g.stride == 1)
            launch_pdl(dwk_strip_kernel<T, V, K, 1, TW, false, ValCoef<V>, ValSrc>, vg.blocks, 256, 0, st, g.hi, g.wi, g.ho, g.wo, g.ci, x, wkc, (const T*)nullptr, items,
                       strips, vg.stride, (T*)z);
        else
            launch_pdl(dwk_strip_kernel<T, V, K, 2, TW, false, ValCoef<V>, ValSrc>, vg.blocks, 256, 0, st, g.hi, g.wi, g.ho, g.wo, g.ci, x, wkc, (const T*)nullptr, items,
                       strips, vg.stride, (T*)z);
    }););
}

void dwk_bwd_data(int dtype, const ConvGeom& g, const GradSrc& dz, const float* wkc, const void* addend, void* dx, cudaStream_t st) {
    const size_t out_e = (size_t)g.n * g.ho * g.wo * g.ci, in_e = (size_t)g.n * g.hi * g.wi * g.ci;
    LaunchScope ls(K_DW_BWD_DATA, ((double)out_e * (grad_needs_z(dz) ? 2 : 1) + (double)in_e * (addend ? 2 : 1)) * esz_(dtype), 2.0 * g.k * g.k * out_e, st);
    DISPATCH_T16(dtype, DISPATCH_K(g.k, {
        constexpr int TW = 4;
        const int strips = (g.wi + TW - 1) / TW, vpr = g.ci / V;
        const size_t items = (size_t)g.n * g.hi * strips * vpr;
        const VecGrid vg = vec_grid(items, vpr, 1);
        if (g.stride == 1)
            launch_pdl(dwk_strip_kernel<T, V, K, 1, TW, true, GradCoef<V>, GradSrc>, vg.blocks, 256, 0, st, g.ho, g.wo, g.hi, g.wi, g.ci, dz, wkc, (const T*)addend, items,
                       strips, vg.stride, (T*)dx);
        else
            launch_pdl(dwk_bwd_data_s2_kernel<T, V, K, TW>, vg.blocks, 256, 0, st, g, dz, wkc, (const T*)addend, items, strips, vg.stride, (T*)dx);
    }););
}

void dwk_bwd_weight(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw, cudaStream_t st) {
    const size_t positions = (size_t)g.n * g.ho * g.wo, out_e = positions * g.ci, in_e = (size_t)g.n * g.hi * g.wi * g.ci;
    const int taps = g.k * g.k;
    int by = 0;
    DISPATCH_T16(dtype, DISPATCH_K(g.k, {
        constexpr int TW = 4;
        const int strips = (g.wo + TW - 1) / TW;
        const size_t total = (size_t)g.n * g.ho * strips;
        const int gx = (g.ci / V + 31) / 32;
        size_t want = ((size_t)4 * sm_count() + gx - 1) / gx;
        const size_t cap = scratch_floats / ((size_t)taps * g.ci);
        if (want > cap) want = cap;
        if (want > (total + 7) / 8) want = (total + 7) / 8;
        if (want < 1) want = 1;
        const size_t spb = (total + want - 1) / want;
        by = (int)((total + spb - 1) / spb);
        LaunchScope ls(K_DW_BWD_WEIGHT, ((double)out_e * (grad_needs_z(dz) ? 2 : 1) + in_e) * esz_(dtype) + 4.0 * taps * g.ci, 2.0 * taps * out_e, st);
        if (g.stride == 1) launch_pdl(dwk_bwd_weight_kernel<T, V, K, 1, TW>, dim3(gx, by), 128, 0, st, g, dz, x, strips, spb, scratch);
        else launch_pdl(dwk_bwd_weight_kernel<T, V, K, 2, TW>, dim3(gx, by), 128, 0, st, g, dz, x, strips, spb, scratch);
    }););
    LaunchScope ls(K_DW_BWD_WEIGHT_FINISH, 4.0 * taps * g.ci * (by + 1), (double)taps * g.ci * by, st);
    launch_pdl(dwk_weight_finish_kernel, (taps * g.ci + 255) / 256, 256, 0, st, (const float*)scratch, by, taps, g.ci, gw);
}

}  // namespace ast
