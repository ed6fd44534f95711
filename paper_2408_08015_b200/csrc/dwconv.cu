// Depthwise 3x3 convolution, NHWC: forward, backward-data and backward-weight.
//
// All three are bandwidth-bound.  A thread owns V consecutive channels (one 16- or 8-byte
// vector) and a horizontal strip of TW output pixels: the per-channel BatchNorm / activation
// coefficients of the producer (forward) or the BatchNorm-backward coefficients (backward) are
// loaded once into registers and applied to every vector on load, an input row is loaded once
// and reused by the three taps and the TW outputs it feeds, and no normalised tensor or dz
// tensor is ever written.  Lanes run along channel vectors, so a warp reads whole pixels.
#include "kernels.h"

namespace ast {
namespace {

constexpr int TW = 4;

// ---- V-wide raw access: (float,4) is 16-byte, (bf16,4) 8-byte ----
template <typename T, int V> struct Raw;
template <> struct Raw<float, 4> {
    static __device__ __forceinline__ void ld(const void* p, size_t e, float* f) {
        float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p) + e);
        f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
    }
    static __device__ __forceinline__ void st(void* p, size_t e, const float* f) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(p) + e) = make_float4(f[0], f[1], f[2], f[3]);
    }
};
template <> struct Raw<__nv_bfloat16, 4> {
    static __device__ __forceinline__ void ld(const void* p, size_t e, float* f) {
        uint2 v = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(p) + e);
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    }
    static __device__ __forceinline__ void st(void* p, size_t e, const float* f) {
        __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]), b = __floats2bfloat162_rn(f[2], f[3]);
        uint2 v = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p) + e) = v;
    }
};

template <int V> __device__ __forceinline__ void ld_coef(const float* p, int c0, float* out) {
#pragma unroll
    for (int q = 0; q < V; q += 4) {
        float4 v = __ldg(reinterpret_cast<const float4*>(p + c0 + q));
        out[q] = v.x; out[q + 1] = v.y; out[q + 2] = v.z; out[q + 3] = v.w;
    }
}

// Reads a forward value: act(raw*scale + shift) with the coefficients held in registers; the
// activation is a pair of bounds and a missing BatchNorm the identity map, so the transform is
// the same instruction stream for every layer configuration.
template <typename T, int V> struct ValLoader {
    const void* p;
    float scale[V], shift[V], lo, hi;
    __device__ __forceinline__ ValLoader(const ValSrc& s, int c0) : p(s.p) {
        if (s.scale) {
            ld_coef<V>(s.scale, c0, scale);
            ld_coef<V>(s.shift, c0, shift);
        } else {
#pragma unroll
            for (int q = 0; q < V; ++q) {
                scale[q] = 1.f;
                shift[q] = 0.f;
            }
        }
        lo = s.act == ACT_NONE ? -INFINITY : 0.f;
        hi = s.act == ACT_RELU6 ? 6.f : INFINITY;
    }
    __device__ __forceinline__ void load(size_t e, float* f) const {
        Raw<T, V>::ld(p, e, f);
#pragma unroll
        for (int q = 0; q < V; ++q) f[q] = fminf(fmaxf(fmaf(f[q], scale[q], shift[q]), lo), hi);
    }
};

// out[n,ho,wo,c] = sum_{r,s} in[n, ho*S-1+r, wo*S-1+s, c] * w[(FLIP ? 8-(3r+s) : 3r+s)][c]  (+ addend)
// Forward: in = x (ValLoader), S = stride.  
template <typename T, int V, int S, bool FLIP, typename LOADER, typename SRC>
__global__ void __launch_bounds__(128) dw_strip_kernel(int n_img, int hi, int wi, int ho, int wo, int c, SRC src, const float* __restrict__ w9c,
                                                       const T* addend, T* out) {
    pdl_wait();
    pdl_launch();
    constexpr int NIN = (TW - 1) * S + 3;
    const int cv = c / V, sw = (wo + TW - 1) / TW;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)n_img * ho * sw * cv) return;
    const int j = (int)(idx % cv);
    size_t sidx = idx / cv;
    const int wo0 = (int)(sidx % sw) * TW;
    size_t t2 = sidx / sw;
    const int oh = (int)(t2 % ho), n = (int)(t2 / ho);
    const int c0 = j * V;
    LOADER ld(src, c0);
    float acc[TW][V];
#pragma unroll
    for (int t = 0; t < TW; ++t)
#pragma unroll
        for (int q = 0; q < V; ++q) acc[t][q] = 0.f;
    const int wi0 = wo0 * S - 1;
    // Halo positions outside the image read a clamped (valid) address and are zeroed afterwards:
    // the body stays straight-line code, so all loads of the three rows can be in flight together.
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int ih = oh * S - 1 + r;
        const bool row_ok = ih >= 0 && ih < hi;
        float xin[NIN][V];
        const size_t rowbase = ((size_t)n * hi + min(max(ih, 0), hi - 1)) * wi;
#pragma unroll
        for (int q2 = 0; q2 < NIN; ++q2) {
            const int iw = wi0 + q2;
            const bool ok = row_ok && iw >= 0 && iw < wi;
            ld.load((rowbase + min(max(iw, 0), wi - 1)) * c + c0, xin[q2]);
#pragma unroll
            for (int q = 0; q < V; ++q) xin[q2][q] = ok ? xin[q2][q] : 0.f;
        }
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            float wv[V];
            ld_coef<V>(w9c + (FLIP ? 8 - (r * 3 + s) : r * 3 + s) * c, c0, wv);
#pragma unroll
            for (int t = 0; t < TW; ++t)
#pragma unroll
                for (int q = 0; q < V; ++q) acc[t][q] = fmaf(xin[t * S + s][q], wv[q], acc[t][q]);
        }
    }
#pragma unroll
    for (int t = 0; t < TW; ++t) {
        if (wo0 + t >= wo) break;
        size_t e = (((size_t)n * ho + oh) * wo + wo0 + t) * c + c0;
        if (addend) {
            float ad[V];
            Raw<T, V>::ld(addend, e, ad);
#pragma unroll
            for (int q = 0; q < V; ++q) acc[t][q] += ad[q];
        }
        Raw<T, V>::st(out, e, acc[t]);
    }
}


// ---------------------------------------------------------------------------------------------
// Rolling-window kernels for stride 1.  A thread owns V channels and a strip TW pixels wide, and
// walks down TH rows: every input row is loaded and transformed once per thread and feeds the
// three output rows it touches from registers, so L1 traffic is 1.5x the input instead of 4.5x;
// the nine per-channel weights come from shared memory; the next row's loads are issued before
// the current row's arithmetic.
template <typename T, int V> struct RawT;
template <> struct RawT<float, 4> { typedef float4 type; };
template <> struct RawT<__nv_bfloat16, 4> { typedef uint2 type; };

template <typename T, int V> __device__ __forceinline__ typename RawT<T, V>::type raw_fetch(const void* p, size_t e);
template <> __device__ __forceinline__ float4 raw_fetch<float, 4>(const void* p, size_t e) {
    return *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p) + e);
}
template <> __device__ __forceinline__ uint2 raw_fetch<__nv_bfloat16, 4>(const void* p, size_t e) {
    return *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(p) + e);
}
__device__ __forceinline__ void raw_decode(const float4& v, float* f) { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
__device__ __forceinline__ void raw_decode(const uint2& v, float* f) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
}

// Split-phase loaders: fetch() only issues the global loads, decode() applies the transform.
// The transforms are branch-free: absent BatchNorm terms take neutral coefficients (scale 1,
// shift 0, k1 1, k2 = k3 0) and the activation is a pair of bounds (ReLU6 0..6, ReLU 0..inf,
// none -inf..inf), so no per-element decision depends on the layer's configuration.
template <typename T, int V> struct ValRoll {
    typedef typename RawT<T, V>::type raw_t;
    struct Raw1 { raw_t a; };
    const void* p;
    float scale[V], shift[V], lo, hi;
    __device__ __forceinline__ ValRoll(const ValSrc& s, int c0) : p(s.p) {
        if (s.scale) {
            ld_coef<V>(s.scale, c0, scale);
            ld_coef<V>(s.shift, c0, shift);
        } else {
#pragma unroll
            for (int q = 0; q < V; ++q) {
                scale[q] = 1.f;
                shift[q] = 0.f;
            }
        }
        lo = s.act == ACT_NONE ? -INFINITY : 0.f;
        hi = s.act == ACT_RELU6 ? 6.f : INFINITY;
    }
    __device__ __forceinline__ Raw1 fetch(size_t e) const { return Raw1{raw_fetch<T, V>(p, e)}; }
    __device__ __forceinline__ void decode(const Raw1& r, bool ok, float* f) const {
        raw_decode(r.a, f);
#pragma unroll
        for (int q = 0; q < V; ++q) {
            const float v = fminf(fmaxf(fmaf(f[q], scale[q], shift[q]), lo), hi);
            f[q] = ok ? v : 0.f;
        }
    }
};
template <typename T, int V> struct GradRoll {
    typedef typename RawT<T, V>::type raw_t;
    struct Raw1 { raw_t a, b; };
    const void* dy;
    const void* z;
    float scale[V], shift[V], k1[V], k2[V], k3[V], lo, hi;
    bool need_z;
    __device__ __forceinline__ GradRoll(const GradSrc& s, int c0) : dy(s.dy), z(s.z), need_z(s.act != ACT_NONE || s.k1 != nullptr) {
#pragma unroll
        for (int q = 0; q < V; ++q) {
            scale[q] = 1.f;
            shift[q] = 0.f;
            k1[q] = 1.f;
            k2[q] = 0.f;
            k3[q] = 0.f;
        }
        if (s.scale) {
            ld_coef<V>(s.scale, c0, scale);
            ld_coef<V>(s.shift, c0, shift);
        }
        if (s.k1) {
            ld_coef<V>(s.k1, c0, k1);
            ld_coef<V>(s.k2, c0, k2);
            ld_coef<V>(s.k3, c0, k3);
        }
        lo = s.act == ACT_NONE ? -INFINITY : 0.f;
        hi = s.act == ACT_RELU6 ? 6.f : INFINITY;
    }
    __device__ __forceinline__ Raw1 fetch(size_t e) const {
        Raw1 r;
        r.a = raw_fetch<T, V>(dy, e);
        r.b = need_z ? raw_fetch<T, V>(z, e) : r.a;
        return r;
    }
    // without z (no activation, no BatchNorm) b == a: pre = dy lies inside (-inf, inf) and the result is dy
    __device__ __forceinline__ void decode(const Raw1& r, bool ok, float* f) const {
        float zz[V];
        raw_decode(r.a, f);
        raw_decode(r.b, zz);
#pragma unroll
        for (int q = 0; q < V; ++q) {
            // lo < pre < hi  <=>  (pre - lo) * (hi - pre) > 0 (exact signs; infinite bounds give +inf,
            // 0 * inf = NaN compares false): the test runs on the FMA pipe and guards one fused multiply-add
            const float pre = fmaf(zz[q], scale[q], shift[q]);
            float d = fmaf(k3[q], zz[q], k2[q]);
            if ((pre - lo) * (hi - pre) > 0.f) d = fmaf(k1[q], f[q], d);
            f[q] = ok ? d : 0.f;
        }
    }
};

// STATS (forward): the kernel also writes the BatchNorm statistics partials of its output,
// stat_partial[block][2][c] = sums of (z - pivot[c]) and (z - pivot[c])^2 over the block's outputs (z as stored, after
// rounding); the threads of a block that own the same channels are combined in thread order.
template <typename T, int V, int TWR, bool FLIP, typename LOADER, typename SRC, bool ADD, bool STATS>
__global__ void __launch_bounds__(128) dw_roll_kernel(int n_img, int h, int w, int c, int th, SRC src, const float* __restrict__ w9c,
                                                      const T* addend, T* out, const float* __restrict__ pivot, float* __restrict__ stat_partial) {
    pdl_launch();
    constexpr int NIN = TWR + 2;
    extern __shared__ float wsm[];            // [9][c], tap order already flipped for the adjoint
    // the weights are not written by the previous kernel in the stream (only the refresh kernel writes them, and it
    // never releases its dependents before it has completed): staging them overlaps that kernel's tail
    for (int i = threadIdx.x; i < 9 * c; i += blockDim.x) {
        int t = i / c, ch = i - t * c;
        wsm[i] = __ldg(w9c + (FLIP ? 8 - t : t) * c + ch);
    }
    __syncthreads();
    pdl_wait();
    const int cv = c / V, sw = (w + TWR - 1) / TWR, nrc = (h + th - 1) / th;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool in_range = idx < (size_t)n_img * nrc * sw * cv;
    if (!STATS && !in_range) return;
    float st1[V], st2[V];
#pragma unroll
    for (int q = 0; q < V; ++q) st1[q] = st2[q] = 0.f;
    if (in_range) {
    const int j = (int)(idx % cv);
    size_t sidx = idx / cv;
    const int wo0 = (int)(sidx % sw) * TWR;
    size_t t2 = sidx / sw;
    const int oh0 = (int)(t2 % nrc) * th, n = (int)(t2 / nrc);
    const int oh1 = min(h, oh0 + th);
    const int c0 = j * V;
    LOADER ld(src, c0);
    typedef typename LOADER::Raw1 Raw1;
    float piv[V];
#pragma unroll
    for (int q = 0; q < V; ++q) piv[q] = STATS ? __ldg(pivot + c0 + q) : 0.f;
    float a0[TWR][V], a1[TWR][V];               // partial sums of output rows ih-1 and ih
#pragma unroll
    for (int t = 0; t < TWR; ++t)
#pragma unroll
        for (int q = 0; q < V; ++q) a0[t][q] = a1[t][q] = 0.f;
    const int wi0 = wo0 - 1;
    int colc[NIN];
    bool colok[NIN];
#pragma unroll
    for (int q2 = 0; q2 < NIN; ++q2) {
        colok[q2] = wi0 + q2 >= 0 && wi0 + q2 < w;
        colc[q2] = min(max(wi0 + q2, 0), w - 1) * c + c0;
    }
    Raw1 nxt[NIN];
    {
        const size_t rb = ((size_t)n * h + max(oh0 - 1, 0)) * w * c;
#pragma unroll
        for (int q2 = 0; q2 < NIN; ++q2) nxt[q2] = ld.fetch(rb + colc[q2]);
    }
    for (int ih = oh0 - 1; ih <= oh1; ++ih) {
        const bool row_ok = ih >= 0 && ih < h;
        float xin[NIN][V];
#pragma unroll
        for (int q2 = 0; q2 < NIN; ++q2) ld.decode(nxt[q2], row_ok && colok[q2], xin[q2]);
        if (ih < oh1) {                        // issue the next row's loads before this row's arithmetic
            const size_t rb = ((size_t)n * h + min(ih + 1, h - 1)) * w * c;
#pragma unroll
            for (int q2 = 0; q2 < NIN; ++q2) nxt[q2] = ld.fetch(rb + colc[q2]);
        }
        float a2[TWR][V];
#pragma unroll
        for (int t = 0; t < TWR; ++t)
#pragma unroll
            for (int q = 0; q < V; ++q) a2[t][q] = 0.f;
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            float w0[V], w1[V], w2[V];
            *reinterpret_cast<float4*>(w0) = *reinterpret_cast<const float4*>(wsm + (0 * 3 + s) * c + c0);
            *reinterpret_cast<float4*>(w1) = *reinterpret_cast<const float4*>(wsm + (1 * 3 + s) * c + c0);
            *reinterpret_cast<float4*>(w2) = *reinterpret_cast<const float4*>(wsm + (2 * 3 + s) * c + c0);
#pragma unroll
            for (int t = 0; t < TWR; ++t)
#pragma unroll
                for (int q = 0; q < V; q += 2) {               // two channels per packed fp32 fused multiply-add
                    const float2 xv = make_float2(xin[t + s][q], xin[t + s][q + 1]);
                    // input row ih is tap row 2 of output row ih-1, tap row 1 of row ih, tap row 0 of row ih+1
                    const float2 r0 = __ffma2_rn(xv, make_float2(w2[q], w2[q + 1]), make_float2(a0[t][q], a0[t][q + 1]));
                    const float2 r1 = __ffma2_rn(xv, make_float2(w1[q], w1[q + 1]), make_float2(a1[t][q], a1[t][q + 1]));
                    const float2 r2 = __ffma2_rn(xv, make_float2(w0[q], w0[q + 1]), make_float2(a2[t][q], a2[t][q + 1]));
                    a0[t][q] = r0.x; a0[t][q + 1] = r0.y;
                    a1[t][q] = r1.x; a1[t][q + 1] = r1.y;
                    a2[t][q] = r2.x; a2[t][q + 1] = r2.y;
                }
        }
        const int orow = ih - 1;
        if (orow >= oh0 && orow < oh1) {
#pragma unroll
            for (int t = 0; t < TWR; ++t) {
                if (wo0 + t < w) {
                    size_t e = (((size_t)n * h + orow) * w + wo0 + t) * c + c0;
                    if (ADD) {
                        float ad[V];
                        Raw<T, V>::ld(addend, e, ad);
#pragma unroll
                        for (int q = 0; q < V; ++q) a0[t][q] += ad[q];
                    }
                    Raw<T, V>::st(out, e, a0[t]);
                    if (STATS) {
#pragma unroll
                        for (int q = 0; q < V; ++q) {
                            const float d = to_f<T>(from_f<T>(a0[t][q])) - piv[q];
                            st1[q] += d;
                            st2[q] = fmaf(d, d, st2[q]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int t = 0; t < TWR; ++t)
#pragma unroll
            for (int q = 0; q < V; ++q) {
                a0[t][q] = a1[t][q];
                a1[t][q] = a2[t][q];
            }
    }
    }
    if (STATS) {
        // thread t owns channel vector (first + t) % cv: vector jv is summed over its threads in thread order
        __syncthreads();                          // the weights in shared memory are no longer needed
        float* red = wsm;                         // [128][2 * V] (the launcher sizes the buffer for both uses)
#pragma unroll
        for (int q = 0; q < V; ++q) {
            red[threadIdx.x * 2 * V + q] = st1[q];
            red[threadIdx.x * 2 * V + V + q] = st2[q];
        }
        __syncthreads();
        const int first = (int)(((size_t)blockIdx.x * blockDim.x) % cv);
        for (int jv = threadIdx.x; jv < cv; jv += blockDim.x) {
            float a1s[V], a2s[V];
#pragma unroll
            for (int q = 0; q < V; ++q) a1s[q] = a2s[q] = 0.f;
            for (int t = (jv - first + cv) % cv; t < (int)blockDim.x; t += cv) {
#pragma unroll
                for (int q = 0; q < V; ++q) {
                    a1s[q] += red[t * 2 * V + q];
                    a2s[q] += red[t * 2 * V + V + q];
                }
            }
            float* dst = stat_partial + (size_t)blockIdx.x * 2 * c + jv * V;
#pragma unroll
            for (int q = 0; q < V; ++q) {
                dst[q] = a1s[q];
                dst[c + q] = a2s[q];
            }
        }
    }
}

// Returns the number of blocks that wrote statistics partials (0: none).
template <typename T, int V, int TWR, bool FLIP, typename LOADER, typename SRC>
int launch_roll(int n, int h, int w, int c, const SRC& src, const float* w9c, const void* addend, void* out, cudaStream_t st,
                const float* pivot = nullptr, float* stat_partial = nullptr, size_t partial_floats = 0) {
    int th = h >= 28 ? 8 : (h >= 14 ? 7 : h);
    size_t total = (size_t)n * ((h + th - 1) / th) * ((w + TWR - 1) / TWR) * (c / V);
    size_t smem = (size_t)9 * c * sizeof(float);
    const unsigned blocks = (unsigned)((total + 127) / 128);
    if (!FLIP && !addend && pivot && stat_partial && (size_t)blocks * 2 * c <= partial_floats) {
        if (smem < (size_t)128 * 2 * V * sizeof(float)) smem = (size_t)128 * 2 * V * sizeof(float);
        launch_pdl(dw_roll_kernel<T, V, TWR, false, LOADER, SRC, false, true>, blocks, 128, smem, st, n, h, w, c, th, src, w9c, (const T*)addend, (T*)out, pivot,
                   stat_partial);
        return (int)blocks;
    }
    if (addend) launch_pdl(dw_roll_kernel<T, V, TWR, FLIP, LOADER, SRC, true, false>, blocks, 128, smem, st, n, h, w, c, th, src, w9c, (const T*)addend, (T*)out,
                           (const float*)nullptr, (float*)nullptr);
    else launch_pdl(dw_roll_kernel<T, V, TWR, FLIP, LOADER, SRC, false, false>, blocks, 128, smem, st, n, h, w, c, th, src, w9c, (const T*)addend, (T*)out,
                    (const float*)nullptr, (float*)nullptr);
    return 0;
}


// Per-thread asynchronous prefetch ring.  A thread copies its own future vectors global -> shared
// with cp.async (one commit group per step) and later reads back only what it copied itself, so
// no barrier is involved: the bytes in flight no longer cost registers and a thread can run
// several rows ahead of its arithmetic.  Slot (stage, load l) of thread t sits at
// ((stage * NL + l) * 128 + t) vectors: consecutive threads are consecutive in shared memory.
template <typename RAW> __device__ __forceinline__ void cp_async_vec(RAW* dst_smem, const void* src) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst_smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2;" ::"r"(d), "l"(src), "n"((int)sizeof(RAW)) : "memory");
}
// same with a 32-bit shared address and a compile-time byte offset (folded into the instruction)
template <int BYTES, int OFF> __device__ __forceinline__ void cp_async_off(uint32_t dst_smem, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0+%2], [%1], %3;" ::"r"(dst_smem), "l"(src), "n"(OFF), "n"(BYTES) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Rolling weight gradient for stride 1: gw[c][r][s] = sum dz[oh][wo] * x[oh-1+r][wo-1+s].
// A thread owns V channels; a work item is a strip TWR wide and `th` rows high.  Walking down the
// input rows ih, it holds dz rows ih-1, ih, ih+1 (zero outside the item's rows) and the x row ih:
// tap row r pairs x row ih with dz row ih+1-r.  Each row of either tensor is loaded and decoded
// once per item; the loads of the next D rows are in flight in the thread's prefetch ring.
template <typename T, int V, int TWR, int D>
__global__ void __launch_bounds__(128) dw_wgrad_roll_kernel(ConvGeom g, GradSrc dzs, ValSrc xs, int cw, int rows, int th, size_t items_per_block,
                                                            float* __restrict__ partial) {
    pdl_wait();
    pdl_launch();
    constexpr int NIN = TWR + 2, NL = NIN + 2 * TWR;
    typedef typename RawT<T, V>::type raw_t;
    extern __shared__ __align__(16) uint8_t dsm[];
    raw_t* ring = reinterpret_cast<raw_t*>(dsm) + threadIdx.x;       // + (stage * NL + l) * 128
    float* red = reinterpret_cast<float*>(dsm);                      // reused after the main loop
    const int cv = g.ci / V;
    const int jl = threadIdx.x % cw, row = threadIdx.x / cw;
    const int j = blockIdx.x * cw + jl;
    const bool active = row < rows && j < cv;
    const int c0 = active ? j * V : 0;
    const int h = g.hi, w = g.wi, c = g.ci;
    const int sw = (w + TWR - 1) / TWR, nrc = (h + th - 1) / th;
    const size_t n_items = (size_t)g.n * nrc * sw;
    const size_t ibeg = (size_t)blockIdx.y * items_per_block, iend = min(n_items, ibeg + items_per_block);
    float acc[9][V];
#pragma unroll
    for (int t = 0; t < 9; ++t)
#pragma unroll
        for (int q = 0; q < V; ++q) acc[t][q] = 0.f;
    if (active) {
        GradRoll<T, V> ldz(dzs, c0);
        ValRoll<T, V> ldx(xs, c0);
        typedef typename GradRoll<T, V>::Raw1 RawZ;
        typedef typename ValRoll<T, V>::Raw1 RawX;
        const T* px = reinterpret_cast<const T*>(xs.p);
        const T* pdy = reinterpret_cast<const T*>(dzs.dy);
        const T* pz = reinterpret_cast<const T*>(dzs.z);
        for (size_t item = ibeg + row; item < iend; item += rows) {
            const int wo0 = (int)(item % sw) * TWR;
            size_t t2 = item / sw;
            const int oh0 = (int)(t2 % nrc) * th, n = (int)(t2 / nrc);
            const int oh1 = min(h, oh0 + th);
            int xcol[NIN], zcol[TWR];
            bool xok[NIN], zok[TWR];
#pragma unroll
            for (int q2 = 0; q2 < NIN; ++q2) {
                const int wi = wo0 - 1 + q2;
                xok[q2] = wi >= 0 && wi < w;
                xcol[q2] = min(max(wi, 0), w - 1) * c + c0;
            }
#pragma unroll
            for (int t = 0; t < TWR; ++t) {
                zok[t] = wo0 + t < w;
                zcol[t] = min(wo0 + t, w - 1) * c + c0;
            }
            // step `ih` consumes x row ih and dz row ih+1 (row addresses clamped into the image)
            auto issue = [&](int ih, int stage) {
                if (ih <= oh1) {
                    const size_t rbx = ((size_t)n * h + min(max(ih, 0), h - 1)) * w * c, rbz = ((size_t)n * h + min(max(ih + 1, 0), h - 1)) * w * c;
                    raw_t* slot = ring + (size_t)stage * NL * 128;
#pragma unroll
                    for (int q2 = 0; q2 < NIN; ++q2) cp_async_vec(slot + q2 * 128, px + rbx + xcol[q2]);
#pragma unroll
                    for (int t = 0; t < TWR; ++t) cp_async_vec(slot + (NIN + t) * 128, pdy + rbz + zcol[t]);
                    if (ldz.need_z) {
#pragma unroll
                        for (int t = 0; t < TWR; ++t) cp_async_vec(slot + (NIN + TWR + t) * 128, pz + rbz + zcol[t]);
                    }
                }
                cp_async_commit();
            };
            float dzm[TWR][V], dz0[TWR][V], dzp[TWR][V];
#pragma unroll
            for (int t = 0; t < TWR; ++t)
#pragma unroll
                for (int q = 0; q < V; ++q) dzm[t][q] = dz0[t][q] = 0.f;
#pragma unroll
            for (int d = 0; d < D; ++d) issue(oh0 - 1 + d, d);
            int stage = 0;
            for (int ih = oh0 - 1; ih <= oh1; ++ih) {
                cp_async_wait<D - 1>();
                const raw_t* slot = ring + (size_t)stage * NL * 128;
                const bool xrow_ok = ih >= 0 && ih < h;
                const bool zrow_ok = ih + 1 >= oh0 && ih + 1 < oh1;
                float xin[NIN][V];
#pragma unroll
                for (int q2 = 0; q2 < NIN; ++q2) {
                    RawX r;
                    r.a = slot[q2 * 128];
                    ldx.decode(r, xrow_ok && xok[q2], xin[q2]);
                }
#pragma unroll
                for (int t = 0; t < TWR; ++t) {
                    RawZ r;
                    r.a = slot[(NIN + t) * 128];
                    r.b = ldz.need_z ? slot[(NIN + TWR + t) * 128] : r.a;
                    ldz.decode(r, zrow_ok && zok[t], dzp[t]);
                }
                issue(ih + D, stage);              // refill the stage just read
                stage = stage + 1 == D ? 0 : stage + 1;
#pragma unroll
                for (int s = 0; s < 3; ++s)
#pragma unroll
                    for (int t = 0; t < TWR; ++t)
#pragma unroll
                        for (int q = 0; q < V; q += 2) {       // two channels per packed fp32 fused multiply-add
                            const float2 xv = make_float2(xin[t + s][q], xin[t + s][q + 1]);
                            const float2 r0 = __ffma2_rn(make_float2(dzp[t][q], dzp[t][q + 1]), xv, make_float2(acc[0 * 3 + s][q], acc[0 * 3 + s][q + 1]));
                            const float2 r1 = __ffma2_rn(make_float2(dz0[t][q], dz0[t][q + 1]), xv, make_float2(acc[1 * 3 + s][q], acc[1 * 3 + s][q + 1]));
                            const float2 r2 = __ffma2_rn(make_float2(dzm[t][q], dzm[t][q + 1]), xv, make_float2(acc[2 * 3 + s][q], acc[2 * 3 + s][q + 1]));
                            acc[0 * 3 + s][q] = r0.x; acc[0 * 3 + s][q + 1] = r0.y;
                            acc[1 * 3 + s][q] = r1.x; acc[1 * 3 + s][q + 1] = r1.y;
                            acc[2 * 3 + s][q] = r2.x; acc[2 * 3 + s][q + 1] = r2.y;
                        }
#pragma unroll
                for (int t = 0; t < TWR; ++t)
#pragma unroll
                    for (int q = 0; q < V; ++q) {
                        dzm[t][q] = dz0[t][q];
                        dz0[t][q] = dzp[t][q];
                    }
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();                               // the ring is now free: reuse it for the block sum
    const int width = cw * V;
    for (int t = 0; t < 9; ++t) {
        if (row < rows) {
#pragma unroll
            for (int q = 0; q < V; ++q) red[row * width + jl * V + q] = acc[t][q];
        }
        __syncthreads();
        for (int e = threadIdx.x; e < width; e += blockDim.x) {
            int ch = blockIdx.x * width + e;
            if (ch < g.ci) {
                float s = 0.f;
                for (int r2 = 0; r2 < rows; ++r2) s += red[r2 * width + e];
                partial[((size_t)blockIdx.y * 9 + t) * g.ci + ch] = s;
            }
        }
        __syncthreads();
    }
}


// Fused backward of a stride-1 depthwise layer: one pass over dy, z and x produces both the input
// gradient and the weight-gradient partials, so the BatchNorm-backward transform of dz is
// evaluated once instead of once per kernel.  A work item is a strip TWR wide over a whole image
// column; a thread owns V channels of it and walks down the rows ih holding dz rows ih-1, ih, ih+1
// (TWR + 2 columns: the strip and one halo column each side) and x row ih:
//   dx[ih][wo0+t]  = sum_{r,s} dz[ih+1-r][wo0+t+1-s] * w[r][s]
//   gw[r][s]      += sum_t dz[ih+1-r][wo0+t] * x[ih][wo0+t-1+s]
// The halo columns of dz feed dx only; their weight-gradient terms belong to the neighbouring strip.
// ADD: the residual gradient `addend` is added to dx (a template parameter: even never-executed
// loads in the inner loop cost issue slots).
template <typename T, int V, int TWR, int D, bool ADD>
__global__ void __launch_bounds__(128, 3) dw_bwd_fused_kernel(ConvGeom g, GradSrc dzs, ValSrc xs, const float* __restrict__ w9c, const T* addend,
                                                           T* dx, int cw, int rows, size_t items_per_block, float* __restrict__ partial) {
    pdl_launch();             // the weights are staged before the dependency wait (see dw_roll_kernel)
    constexpr int NIN = TWR + 2, NL = 3 * NIN;
    typedef typename RawT<T, V>::type raw_t;
    extern __shared__ __align__(16) uint8_t dsm[];
    const int width = cw * V;
    float* wsm = reinterpret_cast<float*>(dsm);                                       // [9][width]
    raw_t* ring = reinterpret_cast<raw_t*>(dsm + (((size_t)9 * width * 4 + 15) & ~(size_t)15)) + threadIdx.x;
    float* red = reinterpret_cast<float*>(ring - threadIdx.x);                        // reused after the main loop
    const int cv = g.ci / V;
    const int jl = threadIdx.x % cw, row = threadIdx.x / cw;
    const int j = blockIdx.x * cw + jl;
    const bool active = row < rows && j < cv;
    const int c0 = active ? j * V : 0;
    const int h = g.hi, w = g.wi, c = g.ci;
    for (int i = threadIdx.x; i < 9 * width; i += blockDim.x) {
        const int t = i / width, ch = blockIdx.x * width + (i - t * width);
        wsm[i] = ch < c ? __ldg(w9c + t * c + ch) : 0.f;
    }
    __syncthreads();
    pdl_wait();
    static_assert(TWR == 2, "the prefetch issue below is written out for four columns");
    constexpr int RB = (int)sizeof(raw_t), SLOT = 128 * RB;          // bytes of one vector / of one load's slots
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
    const int wc = w * c;
    const int sw = (w + TWR - 1) / TWR;
    const size_t n_items = (size_t)g.n * sw;
    const size_t ibeg = (size_t)blockIdx.y * items_per_block, iend = min(n_items, ibeg + items_per_block);
    float acc[9][V];
#pragma unroll
    for (int t = 0; t < 9; ++t)
#pragma unroll
        for (int q = 0; q < V; ++q) acc[t][q] = 0.f;
    if (active) {
        GradRoll<T, V> ldz(dzs, c0);
        ValRoll<T, V> ldx(xs, c0);
        typedef typename GradRoll<T, V>::Raw1 RawZ;
        typedef typename ValRoll<T, V>::Raw1 RawX;
        const T* px = reinterpret_cast<const T*>(xs.p);
        const T* pdy = reinterpret_cast<const T*>(dzs.dy);
        const T* pz = reinterpret_cast<const T*>(dzs.z);
        const float* wl = wsm + jl * V;
        for (size_t item = ibeg + row; item < iend; item += rows) {
            const int wo0 = (int)(item % sw) * TWR, n = (int)(item / sw);
            int col[NIN];
            bool cok[NIN];
#pragma unroll
            for (int q2 = 0; q2 < NIN; ++q2) {
                const int wi = wo0 - 1 + q2;
                cok[q2] = wi >= 0 && wi < w;
                col[q2] = min(max(wi, 0), w - 1) * c + c0;
            }
            // step ih consumes x row ih and dz row ih+1 (row addresses clamped into the image)
            const T* px_n = px + (size_t)n * h * wc;
            const T* pdy_n = pdy + (size_t)n * h * wc;
            const T* pz_n = pz + (size_t)n * h * wc;
            auto issue = [&](int ih, int stage) {
                if (ih < h) {
                    const T* rx = px_n + max(ih, 0) * wc;
                    const int zoff = min(ih + 1, h - 1) * wc;
                    const T* rdy = pdy_n + zoff;
                    const T* rz = pz_n + zoff;
                    const uint32_t s0 = ring_s + (uint32_t)stage * (uint32_t)(NL * SLOT);
                    cp_async_off<RB, 0 * SLOT>(s0, rx + col[0]);
                    cp_async_off<RB, 1 * SLOT>(s0, rx + col[1]);
                    cp_async_off<RB, 2 * SLOT>(s0, rx + col[2]);
                    cp_async_off<RB, 3 * SLOT>(s0, rx + col[3]);
                    cp_async_off<RB, 4 * SLOT>(s0, rdy + col[0]);
                    cp_async_off<RB, 5 * SLOT>(s0, rdy + col[1]);
                    cp_async_off<RB, 6 * SLOT>(s0, rdy + col[2]);
                    cp_async_off<RB, 7 * SLOT>(s0, rdy + col[3]);
                    if (ldz.need_z) {
                        cp_async_off<RB, 8 * SLOT>(s0, rz + col[0]);
                        cp_async_off<RB, 9 * SLOT>(s0, rz + col[1]);
                        cp_async_off<RB, 10 * SLOT>(s0, rz + col[2]);
                        cp_async_off<RB, 11 * SLOT>(s0, rz + col[3]);
                    }
                }
                cp_async_commit();
            };
            float dzm[NIN][V], dz0[NIN][V], dzp[NIN][V];
#pragma unroll
            for (int q2 = 0; q2 < NIN; ++q2)
#pragma unroll
                for (int q = 0; q < V; ++q) dzm[q2][q] = dz0[q2][q] = 0.f;
#pragma unroll
            for (int d = 0; d < D; ++d) issue(-1 + d, d);
            int stage = 0;
            for (int ih = -1; ih < h; ++ih) {
                cp_async_wait<D - 1>();
                const raw_t* slot = ring + (size_t)stage * NL * 128;
                const bool xrow_ok = ih >= 0, zrow_ok = ih + 1 < h;
                float xin[NIN][V];
#pragma unroll
                for (int q2 = 0; q2 < NIN; ++q2) {
                    RawX r;
                    r.a = slot[q2 * 128];
                    ldx.decode(r, xrow_ok && cok[q2], xin[q2]);
                }
#pragma unroll
                for (int q2 = 0; q2 < NIN; ++q2) {
                    RawZ r;
                    r.a = slot[(NIN + q2) * 128];
                    r.b = ldz.need_z ? slot[(2 * NIN + q2) * 128] : r.a;
                    ldz.decode(r, zrow_ok && cok[q2], dzp[q2]);
                }
                issue(ih + D, stage);              // refill the stage just read
                stage = stage + 1 == D ? 0 : stage + 1;
                float ad[TWR][V];
                const size_t orow = (((size_t)n * h + max(ih, 0)) * w + wo0) * c + c0;
                if (ADD && ih >= 0) {
#pragma unroll
                    for (int t = 0; t < TWR; ++t)
                        if (wo0 + t < w) Raw<T, V>::ld(addend, orow + (size_t)t * c, ad[t]);
                }
                float o[TWR][V];
#pragma unroll
                for (int t = 0; t < TWR; ++t)
#pragma unroll
                    for (int q = 0; q < V; ++q) o[t][q] = 0.f;
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    float w0[V], w1[V], w2[V];
                    *reinterpret_cast<float4*>(w0) = *reinterpret_cast<const float4*>(wl + (0 * 3 + s) * width);
                    *reinterpret_cast<float4*>(w1) = *reinterpret_cast<const float4*>(wl + (1 * 3 + s) * width);
                    *reinterpret_cast<float4*>(w2) = *reinterpret_cast<const float4*>(wl + (2 * 3 + s) * width);
                    // two channels per instruction (packed fp32 fused multiply-add)
#pragma unroll
                    for (int t = 0; t < TWR; ++t)
#pragma unroll
                        for (int q = 0; q < V; q += 2) {
                            float2 oo = make_float2(o[t][q], o[t][q + 1]);
                            oo = __ffma2_rn(make_float2(dzp[t + 2 - s][q], dzp[t + 2 - s][q + 1]), make_float2(w0[q], w0[q + 1]), oo);
                            oo = __ffma2_rn(make_float2(dz0[t + 2 - s][q], dz0[t + 2 - s][q + 1]), make_float2(w1[q], w1[q + 1]), oo);
                            oo = __ffma2_rn(make_float2(dzm[t + 2 - s][q], dzm[t + 2 - s][q + 1]), make_float2(w2[q], w2[q + 1]), oo);
                            o[t][q] = oo.x;
                            o[t][q + 1] = oo.y;
                            const float2 xv = make_float2(xin[t + s][q], xin[t + s][q + 1]);
                            float2 a0 = make_float2(acc[0 * 3 + s][q], acc[0 * 3 + s][q + 1]);
                            float2 a1 = make_float2(acc[1 * 3 + s][q], acc[1 * 3 + s][q + 1]);
                            float2 a2 = make_float2(acc[2 * 3 + s][q], acc[2 * 3 + s][q + 1]);
                            a0 = __ffma2_rn(make_float2(dzp[t + 1][q], dzp[t + 1][q + 1]), xv, a0);
                            a1 = __ffma2_rn(make_float2(dz0[t + 1][q], dz0[t + 1][q + 1]), xv, a1);
                            a2 = __ffma2_rn(make_float2(dzm[t + 1][q], dzm[t + 1][q + 1]), xv, a2);
                            acc[0 * 3 + s][q] = a0.x; acc[0 * 3 + s][q + 1] = a0.y;
                            acc[1 * 3 + s][q] = a1.x; acc[1 * 3 + s][q + 1] = a1.y;
                            acc[2 * 3 + s][q] = a2.x; acc[2 * 3 + s][q + 1] = a2.y;
                        }
                }
                if (ih >= 0) {
#pragma unroll
                    for (int t = 0; t < TWR; ++t) {
                        if (wo0 + t < w) {
                            if (ADD) {
#pragma unroll
                                for (int q = 0; q < V; ++q) o[t][q] += ad[t][q];
                            }
                            Raw<T, V>::st(dx, orow + (size_t)t * c, o[t]);
                        }
                    }
                }
#pragma unroll
                for (int q2 = 0; q2 < NIN; ++q2)
#pragma unroll
                    for (int q = 0; q < V; ++q) {
                        dzm[q2][q] = dz0[q2][q];
                        dz0[q2][q] = dzp[q2][q];
                    }
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();                               // the ring is now free: reuse it for the block sum
    for (int t = 0; t < 9; ++t) {
        if (row < rows) {
#pragma unroll
            for (int q = 0; q < V; ++q) red[row * width + jl * V + q] = acc[t][q];
        }
        __syncthreads();
        for (int e = threadIdx.x; e < width; e += blockDim.x) {
            int ch = blockIdx.x * width + e;
            if (ch < g.ci) {
                float s = 0.f;
                for (int r2 = 0; r2 < rows; ++r2) s += red[r2 * width + e];
                partial[((size_t)blockIdx.y * 9 + t) * g.ci + ch] = s;
            }
        }
        __syncthreads();
    }
}


// ---------------------------------------------------------------------------------------------
// Stride-2 backward kernels, rolling over the rows of dz.
// Forward: z(ho,wo) = sum_{r,s} x(2ho-1+r, 2wo-1+s) w(r,s).  Hence an even input row 2i receives
// only tap row 1 of dz row i; an odd input row 2i+1 receives tap row 2 of dz row i and tap row 0
// of dz row i+1; columns likewise.  A thread owns V channels and TWZ columns of dz (plus one
// halo column), walks down the dz rows keeping rows i and i+1, and writes the two input rows
// 2i, 2i+1 (2*TWZ columns each).  Every dz element is loaded and transformed once per thread.
template <typename T, int V, int TWZ, bool ADD>
__global__ void __launch_bounds__(128) dw_bwd_data_s2_kernel(ConvGeom g, GradSrc dzs, const float* __restrict__ w9c, int th, const T* addend, T* dx) {
    pdl_launch();             // the weights are staged before the dependency wait (see dw_roll_kernel)
    extern __shared__ float wsm[];            // [9][c]
    const int c = g.ci, H = g.hi, W = g.wi, Ho = g.ho, Wo = g.wo;
    for (int i = threadIdx.x; i < 9 * c; i += blockDim.x) wsm[i] = __ldg(w9c + i);
    __syncthreads();
    pdl_wait();
    const int cv = c / V;
    const int nrowz = (H + 1) / 2, ncolz = (W + 1) / 2;              // dz rows / columns that own input rows / columns
    const int swz = (ncolz + TWZ - 1) / TWZ, nrc = (nrowz + th - 1) / th;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)g.n * nrc * swz * cv) return;
    const int j = (int)(idx % cv);
    size_t sidx = idx / cv;
    const int jz0 = (int)(sidx % swz) * TWZ;
    size_t t2 = sidx / swz;
    const int i0 = (int)(t2 % nrc) * th, n = (int)(t2 / nrc);
    const int i1 = min(nrowz, i0 + th);
    const int c0 = j * V;
    GradRoll<T, V> ld(dzs, c0);
    typedef typename GradRoll<T, V>::Raw1 Raw1;
    float wt[9][V];
#pragma unroll
    for (int t = 0; t < 9; ++t) *reinterpret_cast<float4*>(wt[t]) = *reinterpret_cast<const float4*>(wsm + t * c + c0);
    int zcol[TWZ + 1];
    bool zok[TWZ + 1];
#pragma unroll
    for (int q2 = 0; q2 <= TWZ; ++q2) {
        zok[q2] = jz0 + q2 < Wo;
        zcol[q2] = min(jz0 + q2, Wo - 1) * c + c0;
    }
    float cur[TWZ + 1][V], nxt[TWZ + 1][V];
    Raw1 raw[TWZ + 1];
    {   // dz row i0 decoded into cur; raw of row i0+1 requested
        const size_t rb = ((size_t)n * Ho + min(i0, Ho - 1)) * Wo * c;
#pragma unroll
        for (int q2 = 0; q2 <= TWZ; ++q2) raw[q2] = ld.fetch(rb + zcol[q2]);
#pragma unroll
        for (int q2 = 0; q2 <= TWZ; ++q2) ld.decode(raw[q2], zok[q2] && i0 < Ho, cur[q2]);
        const size_t rb1 = ((size_t)n * Ho + min(i0 + 1, Ho - 1)) * Wo * c;
#pragma unroll
        for (int q2 = 0; q2 <= TWZ; ++q2) raw[q2] = ld.fetch(rb1 + zcol[q2]);
    }
    for (int i = i0; i < i1; ++i) {
#pragma unroll
        for (int q2 = 0; q2 <= TWZ; ++q2) ld.decode(raw[q2], zok[q2] && i + 1 < Ho, nxt[q2]);
        if (i + 1 < i1) {
            const size_t rb = ((size_t)n * Ho + min(i + 2, Ho - 1)) * Wo * c;
#pragma unroll
            for (int q2 = 0; q2 <= TWZ; ++q2) raw[q2] = ld.fetch(rb + zcol[q2]);
        }
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            const int hi = 2 * i + a;
            if (hi >= H) continue;
#pragma unroll
            for (int t = 0; t < TWZ; ++t) {
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    const int wi = 2 * (jz0 + t) + b;
                    if (wi >= W) continue;
                    float o[V];
#pragma unroll
                    for (int q = 0; q < V; ++q) {
                        float v;
                        if (a == 0 && b == 0) {
                            v = cur[t][q] * wt[4][q];
                        } else if (a == 0) {
                            v = fmaf(cur[t][q], wt[5][q], cur[t + 1][q] * wt[3][q]);
                        } else if (b == 0) {
                            v = fmaf(cur[t][q], wt[7][q], nxt[t][q] * wt[1][q]);
                        } else {
                            v = fmaf(cur[t][q], wt[8][q], fmaf(cur[t + 1][q], wt[6][q], fmaf(nxt[t][q], wt[2][q], nxt[t + 1][q] * wt[0][q])));
                        }
                        o[q] = v;
                    }
                    const size_t e = (((size_t)n * H + hi) * W + wi) * c + c0;
                    if (ADD) {
                        float ad[V];
                        Raw<T, V>::ld(addend, e, ad);
#pragma unroll
                        for (int q = 0; q < V; ++q) o[q] += ad[q];
                    }
                    Raw<T, V>::st(dx, e, o);
                }
            }
        }
#pragma unroll
        for (int q2 = 0; q2 <= TWZ; ++q2)
#pragma unroll
            for (int q = 0; q < V; ++q) cur[q2][q] = nxt[q2][q];
    }
}

// Stride-2 weight gradient: gw[c][r][s] = sum dz(ho,wo) x(2ho-1+r, 2wo-1+s).  A work item is TWZ
// columns by `th` rows of dz; walking down the dz rows, x row 2ho+1 of one step is x row 2ho'-1 of
// the next, so each x row is loaded and transformed once.
template <typename T, int V, int TWZ>
__global__ void __launch_bounds__(128) dw_wgrad_s2_kernel(ConvGeom g, GradSrc dzs, ValSrc xs, int cw, int rows, int th, size_t items_per_block,
                                                          float* __restrict__ partial) {
    pdl_wait();
    pdl_launch();
    constexpr int NX = 2 * TWZ + 1;
    extern __shared__ float red[];
    const int cv = g.ci / V;
    const int jl = threadIdx.x % cw, row = threadIdx.x / cw;
    const int j = blockIdx.x * cw + jl;
    const bool active = row < rows && j < cv;
    const int c0 = active ? j * V : 0;
    const int H = g.hi, W = g.wi, Ho = g.ho, Wo = g.wo, c = g.ci;
    const int swz = (Wo + TWZ - 1) / TWZ, nrc = (Ho + th - 1) / th;
    const size_t n_items = (size_t)g.n * nrc * swz;
    const size_t ibeg = (size_t)blockIdx.y * items_per_block, iend = min(n_items, ibeg + items_per_block);
    float acc[9][V];
#pragma unroll
    for (int t = 0; t < 9; ++t)
#pragma unroll
        for (int q = 0; q < V; ++q) acc[t][q] = 0.f;
    if (active) {
        GradRoll<T, V> ldz(dzs, c0);
        ValRoll<T, V> ldx(xs, c0);
        typedef typename GradRoll<T, V>::Raw1 RawZ;
        typedef typename ValRoll<T, V>::Raw1 RawX;
        for (size_t item = ibeg + row; item < iend; item += rows) {
            const int wo0 = (int)(item % swz) * TWZ;
            size_t t2 = item / swz;
            const int oh0 = (int)(t2 % nrc) * th, n = (int)(t2 / nrc);
            const int oh1 = min(Ho, oh0 + th);
            int xcol[NX], zcol[TWZ];
            bool xok[NX], zok[TWZ];
#pragma unroll
            for (int q2 = 0; q2 < NX; ++q2) {
                const int wi = 2 * wo0 - 1 + q2;
                xok[q2] = wi >= 0 && wi < W;
                xcol[q2] = min(max(wi, 0), W - 1) * c + c0;
            }
#pragma unroll
            for (int t = 0; t < TWZ; ++t) {
                zok[t] = wo0 + t < Wo;
                zcol[t] = min(wo0 + t, Wo - 1) * c + c0;
            }
            float xp[NX][V];     // x row 2ho-1
            {
                const int ih = 2 * oh0 - 1;
                const size_t rb = ((size_t)n * H + max(ih, 0)) * W * c;
#pragma unroll
                for (int q2 = 0; q2 < NX; ++q2) {
                    RawX r = ldx.fetch(rb + xcol[q2]);
                    ldx.decode(r, ih >= 0 && xok[q2], xp[q2]);
                }
            }
            RawX nxa[NX], nxb[NX];
            RawZ nz[TWZ];
            {
                const size_t ra = ((size_t)n * H + min(2 * oh0, H - 1)) * W * c, rb = ((size_t)n * H + min(2 * oh0 + 1, H - 1)) * W * c;
                const size_t rz = ((size_t)n * Ho + oh0) * Wo * c;
#pragma unroll
                for (int q2 = 0; q2 < NX; ++q2) {
                    nxa[q2] = ldx.fetch(ra + xcol[q2]);
                    nxb[q2] = ldx.fetch(rb + xcol[q2]);
                }
#pragma unroll
                for (int t = 0; t < TWZ; ++t) nz[t] = ldz.fetch(rz + zcol[t]);
            }
            for (int oh = oh0; oh < oh1; ++oh) {
                float xa[NX][V], xb[NX][V], dv[TWZ][V];
#pragma unroll
                for (int q2 = 0; q2 < NX; ++q2) {
                    ldx.decode(nxa[q2], 2 * oh < H && xok[q2], xa[q2]);
                    ldx.decode(nxb[q2], 2 * oh + 1 < H && xok[q2], xb[q2]);
                }
#pragma unroll
                for (int t = 0; t < TWZ; ++t) ldz.decode(nz[t], zok[t], dv[t]);
                if (oh + 1 < oh1) {
                    const size_t ra = ((size_t)n * H + min(2 * oh + 2, H - 1)) * W * c, rb = ((size_t)n * H + min(2 * oh + 3, H - 1)) * W * c;
                    const size_t rz = ((size_t)n * Ho + oh + 1) * Wo * c;
#pragma unroll
                    for (int q2 = 0; q2 < NX; ++q2) {
                        nxa[q2] = ldx.fetch(ra + xcol[q2]);
                        nxb[q2] = ldx.fetch(rb + xcol[q2]);
                    }
#pragma unroll
                    for (int t = 0; t < TWZ; ++t) nz[t] = ldz.fetch(rz + zcol[t]);
                }
#pragma unroll
                for (int s = 0; s < 3; ++s)
#pragma unroll
                    for (int t = 0; t < TWZ; ++t)
#pragma unroll
                        for (int q = 0; q < V; ++q) {
                            acc[0 * 3 + s][q] = fmaf(dv[t][q], xp[2 * t + s][q], acc[0 * 3 + s][q]);
                            acc[1 * 3 + s][q] = fmaf(dv[t][q], xa[2 * t + s][q], acc[1 * 3 + s][q]);
                            acc[2 * 3 + s][q] = fmaf(dv[t][q], xb[2 * t + s][q], acc[2 * 3 + s][q]);
                        }
#pragma unroll
                for (int q2 = 0; q2 < NX; ++q2)
#pragma unroll
                    for (int q = 0; q < V; ++q) xp[q2][q] = xb[q2][q];
            }
        }
    }
    const int width = cw * V;
    for (int t = 0; t < 9; ++t) {
        if (row < rows) {
#pragma unroll
            for (int q = 0; q < V; ++q) red[row * width + jl * V + q] = acc[t][q];
        }
        __syncthreads();
        for (int e = threadIdx.x; e < width; e += blockDim.x) {
            int ch = blockIdx.x * width + e;
            if (ch < g.ci) {
                float s = 0.f;
                for (int r2 = 0; r2 < rows; ++r2) s += red[r2 * width + e];
                partial[((size_t)blockIdx.y * 9 + t) * g.ci + ch] = s;
            }
        }
        __syncthreads();
    }
}

// gw[c][t] = sum_b partial[b][t][c]; one warp per (t, c): lanes stride over the blocks
__global__ void __launch_bounds__(128) dw_bwd_weight_finish(const float* __restrict__ partial, int blocks, int c_total, float* __restrict__ gw) {
    pdl_wait();
    pdl_launch();
    int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (i >= 9 * c_total) return;
    int t = i / c_total, c = i % c_total;
    float s = 0.f;
    for (int b0 = threadIdx.x & 31; b0 < blocks; b0 += 32 * 8) {   // eight loads in flight, fixed addition order
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = (b0 + 32 * u < blocks) ? partial[((size_t)(b0 + 32 * u) * 9 + t) * c_total + c] : 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) s += v[u];
    }
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) gw[c * 9 + t] = s;
}

double esz(int dtype) { return dtype == 0 ? 4.0 : 2.0; }
double grad_src_bytes(const GradSrc& d, double elems, int dtype) { return elems * esz(dtype) * ((d.act != ACT_NONE || d.k1) ? 2.0 : 1.0); }

template <typename T, int V, int S, bool FLIP, typename LOADER, typename SRC>
void launch_strip(int n, int hi, int wi, int ho, int wo, int c, const SRC& src, const float* w9c, const void* addend, void* out, cudaStream_t st) {
    size_t total = (size_t)n * ho * ((wo + TW - 1) / TW) * (c / V);
    launch_pdl(dw_strip_kernel<T, V, S, FLIP, LOADER, SRC>, (unsigned)((total + 127) / 128), 128, 0, st, n, hi, wi, ho, wo, c, src, w9c, (const T*)addend, (T*)out);
}

}  // namespace

int dw_fwd(int dtype, const ConvGeom& g, const ValSrc& x, const float* w9c, void* z, const float* pivot, float* partial, size_t partial_floats,
           cudaStream_t st) {
    double in_e = (double)g.n * g.hi * g.wi * g.ci, out_e = (double)g.n * g.ho * g.wo * g.ci;
    LaunchScope ls(K_DW_FWD, (in_e + out_e) * esz(dtype) + 36.0 * g.ci, 18.0 * out_e, st);
    using B = __nv_bfloat16;
    if (dtype == 0) {
        if (g.stride == 1) return launch_roll<float, 4, 4, false, ValRoll<float, 4>, ValSrc>(g.n, g.hi, g.wi, g.ci, x, w9c, nullptr, z, st, pivot, partial, partial_floats);
        launch_strip<float, 4, 2, false, ValLoader<float, 4>, ValSrc>(g.n, g.hi, g.wi, g.ho, g.wo, g.ci, x, w9c, nullptr, z, st);
    } else {
        if (g.stride == 1) return launch_roll<B, 4, 4, false, ValRoll<B, 4>, ValSrc>(g.n, g.hi, g.wi, g.ci, x, w9c, nullptr, z, st, pivot, partial, partial_floats);
        launch_strip<B, 4, 2, false, ValLoader<B, 4>, ValSrc>(g.n, g.hi, g.wi, g.ho, g.wo, g.ci, x, w9c, nullptr, z, st);
    }
    return 0;
}

void dw_bwd_data(int dtype, const ConvGeom& g, const GradSrc& dz, const float* w9c, const void* addend, void* dx, cudaStream_t st) {
    double in_e = (double)g.n * g.hi * g.wi * g.ci, out_e = (double)g.n * g.ho * g.wo * g.ci;
    LaunchScope ls(K_DW_BWD_DATA, grad_src_bytes(dz, out_e, dtype) + in_e * esz(dtype) * (addend ? 2.0 : 1.0) + 36.0 * g.ci, 18.0 * out_e, st);
    using B = __nv_bfloat16;
    if (g.stride == 1) {
        // the adjoint of a stride-1 3x3 correlation is the correlation of dz with the flipped kernel
        if (dtype == 0) launch_roll<float, 4, 4, true, GradRoll<float, 4>, GradSrc>(g.n, g.hi, g.wi, g.ci, dz, w9c, addend, dx, st);
        else launch_roll<B, 4, 2, true, GradRoll<B, 4>, GradSrc>(g.n, g.hi, g.wi, g.ci, dz, w9c, addend, dx, st);
    } else {
        constexpr int TWZ = 2;
        const int nrowz = (g.hi + 1) / 2, ncolz = (g.wi + 1) / 2;
        const int th = nrowz >= 14 ? 7 : nrowz;
        size_t total = (size_t)g.n * ((nrowz + th - 1) / th) * ((ncolz + TWZ - 1) / TWZ) * (g.ci / 4);
        size_t smem = (size_t)9 * g.ci * sizeof(float);
        const unsigned blocks = (unsigned)((total + 127) / 128);
        if (dtype == 0) {
            if (addend) launch_pdl(dw_bwd_data_s2_kernel<float, 4, TWZ, true>, blocks, 128, smem, st, g, dz, w9c, th, (const float*)addend, (float*)dx);
            else launch_pdl(dw_bwd_data_s2_kernel<float, 4, TWZ, false>, blocks, 128, smem, st, g, dz, w9c, th, (const float*)addend, (float*)dx);
        } else {
            if (addend) launch_pdl(dw_bwd_data_s2_kernel<B, 4, TWZ, true>, blocks, 128, smem, st, g, dz, w9c, th, (const B*)addend, (B*)dx);
            else launch_pdl(dw_bwd_data_s2_kernel<B, 4, TWZ, false>, blocks, 128, smem, st, g, dz, w9c, th, (const B*)addend, (B*)dx);
        }
    }
}

void dw_bwd_weight(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw,
                   cudaStream_t st) {
    constexpr int TWR = 2;
    const int V = 4;
    const int cv = g.ci / V;
    const int parts = (cv + 47) / 48;              // channel-vector columns per block: an even split, at most 48
    const int cw = (cv + parts - 1) / parts;
    const int rows = 128 / cw;
    const int gx = (cv + cw - 1) / cw;
    const int sw = (g.wo + TWR - 1) / TWR;
    const size_t cap = scratch_floats / ((size_t)9 * g.ci);
    double in_e = (double)g.n * g.hi * g.wi * g.ci, out_e = (double)g.n * g.ho * g.wo * g.ci;
    size_t by;
    if (g.stride == 1) {
        // Long items (whole image columns when the batch gives enough of them) keep the prefetch
        // ring full; all blocks are resident at once, so there is no partial last wave.
        const size_t resident = 3 * (size_t)sm_count();
        int th = g.ho;
        while (th > 7 && (size_t)g.n * ((g.ho + th - 1) / th) * sw * gx < (size_t)rows * 2 * sm_count()) th = (th + 1) / 2;
        const size_t n_items = (size_t)g.n * ((g.ho + th - 1) / th) * sw;
        by = (n_items + rows - 1) / rows;
        if (by * gx > resident) by = resident / gx;
        if (by > cap) by = cap;
        if (by < 1) by = 1;
        const size_t ipb = (n_items + by - 1) / by;
        by = (n_items + ipb - 1) / ipb;
        dim3 grid(gx, (unsigned)by);
        LaunchScope ls(K_DW_BWD_WEIGHT, grad_src_bytes(dz, out_e, dtype) + in_e * esz(dtype) + 36.0 * g.ci, 18.0 * out_e, st);
        constexpr int NL = TWR + 2 + 2 * TWR;
        if (dtype == 0) {
            constexpr int D = 2;
            launch_pdl(dw_wgrad_roll_kernel<float, 4, TWR, D>, grid, 128, (size_t)D * NL * 128 * 16, st, g, dz, x, cw, rows, th, ipb, scratch);
        } else {
            constexpr int D = 4;
            launch_pdl(dw_wgrad_roll_kernel<__nv_bfloat16, 4, TWR, D>, grid, 128, (size_t)D * NL * 128 * 8, st, g, dz, x, cw, rows, th, ipb, scratch);
        }
    } else {
        const int th = g.ho >= 28 ? 8 : (g.ho >= 14 ? 7 : g.ho);      // rows of dz per work item
        const int nrc = (g.ho + th - 1) / th;
        const size_t n_items = (size_t)g.n * nrc * sw;
        by = (8 * sm_count() + gx - 1) / gx;
        const size_t max_by = (n_items + (size_t)rows - 1) / (size_t)rows;
        if (by > max_by) by = max_by;
        if (by > cap) by = cap;
        if (by < 1) by = 1;
        const size_t ipb = (n_items + by - 1) / by;
        by = (n_items + ipb - 1) / ipb;
        const size_t smem = (size_t)rows * cw * V * sizeof(float);
        dim3 grid(gx, (unsigned)by);
        LaunchScope ls(K_DW_BWD_WEIGHT, grad_src_bytes(dz, out_e, dtype) + in_e * esz(dtype) + 36.0 * g.ci, 18.0 * out_e, st);
        if (dtype == 0) launch_pdl(dw_wgrad_s2_kernel<float, 4, TWR>, grid, 128, smem, st, g, dz, x, cw, rows, th, ipb, scratch);
        else launch_pdl(dw_wgrad_s2_kernel<__nv_bfloat16, 4, TWR>, grid, 128, smem, st, g, dz, x, cw, rows, th, ipb, scratch);
    }
    LaunchScope ls(K_DW_BWD_WEIGHT_FINISH, 36.0 * g.ci * (by + 1), 9.0 * g.ci * by, st);
    launch_pdl(dw_bwd_weight_finish, (9 * g.ci + 3) / 4, 128, 0, st, scratch, (int)by, g.ci, gw);
}

bool dw_bwd_fused(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, const float* w9c, const void* addend, void* dx,
                  float* scratch, size_t scratch_floats, float* gw, cudaStream_t st) {
    constexpr int TWR = 2, V = 4, D = 4, NL = 3 * (TWR + 2);
    if (dtype != 1 || g.stride != 1 || g.ci % V) return false;
    const int cv = g.ci / V;
    const int parts = (cv + 47) / 48;
    const int cw = (cv + parts - 1) / parts;
    const int rows = 128 / cw;
    const int gx = (cv + cw - 1) / cw;
    const int sw = (g.wo + TWR - 1) / TWR;
    const size_t n_items = (size_t)g.n * sw;
    // whole image columns per thread: worth it only when that still gives every SM a few warps
    if (n_items * gx < (size_t)rows * 2 * sm_count()) return false;
    const size_t cap = scratch_floats / ((size_t)9 * g.ci);
    const size_t resident = 3 * (size_t)sm_count();              // three blocks per SM: all blocks run at once, no partial last wave
    size_t by = (n_items + rows - 1) / rows;
    if (by * gx > resident) by = resident / gx;
    if (by > cap) by = cap;
    if (by < 1) return false;
    const size_t ipb = (n_items + by - 1) / by;
    by = (n_items + ipb - 1) / ipb;
    const size_t smem = (((size_t)9 * cw * V * 4 + 15) & ~(size_t)15) + (size_t)D * NL * 128 * 8;
    smem_limit_once<201 + V * 10000 + TWR * 1000 + D * 100>(dw_bwd_fused_kernel<__nv_bfloat16, V, TWR, D, true>, 96 * 1024);
    smem_limit_once<202 + V * 10000 + TWR * 1000 + D * 100>(dw_bwd_fused_kernel<__nv_bfloat16, V, TWR, D, false>, 96 * 1024);
    double e = (double)g.n * g.hi * g.wi * g.ci;
    {
        LaunchScope ls(K_DW_BWD_FUSED, grad_src_bytes(dz, e, dtype) + e * 2.0 * (addend ? 3.0 : 2.0) + 36.0 * g.ci, 36.0 * e, st);
        dim3 grid(gx, (unsigned)by);
        if (addend) launch_pdl(dw_bwd_fused_kernel<__nv_bfloat16, V, TWR, D, true>, grid, 128, smem, st, g, dz, x, w9c, (const __nv_bfloat16*)addend, (__nv_bfloat16*)dx, cw,
                                                                            rows, ipb, scratch);
        else launch_pdl(dw_bwd_fused_kernel<__nv_bfloat16, V, TWR, D, false>, grid, 128, smem, st, g, dz, x, w9c, (const __nv_bfloat16*)addend, (__nv_bfloat16*)dx, cw,
                                                                            rows, ipb, scratch);
    }
    LaunchScope ls(K_DW_BWD_WEIGHT_FINISH, 36.0 * g.ci * (by + 1), 9.0 * g.ci * by, st);
    launch_pdl(dw_bwd_weight_finish, (9 * g.ci + 3) / 4, 128, 0, st, scratch, (int)by, g.ci, gw);
    return true;
}

}  // namespace ast
