// Shared device helpers of the stage kernels: storage-type conversion, the descriptors by
// which a kernel reads a forward value or a conv-output gradient "on load", reductions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ast {

enum { ACT_NONE = 0, ACT_RELU6 = 1, ACT_RELU = 2 };

// A forward value as consumers read it.  A conv->BN->activation chain is never written out in
// normalised form: consumers read the raw conv output z and apply  act(z*scale[c] + shift[c])
// while loading.  scale == nullptr means the tensor holds the value itself.
struct ValSrc {
    const void* p;
    const float* scale;
    const float* shift;
    int act;
};

// Gradient w.r.t. a raw conv output z, formed while loading from the gradient dy w.r.t. the
// chain's output value:  pre = z*scale+shift;  dpre = dy * [pre inside the activation's linear
// region];  dz = k1*dpre + k2 + k3*z  (BatchNorm backward with the two per-channel sums folded
// into k2, k3).  k1 == nullptr: no BatchNorm, dz = dpre.  act == 0 and scale == nullptr: dz = dy.
struct GradSrc {
    const void* dy;
    const void* z;
    const float* scale;
    const float* shift;
    const float* k1;
    const float* k2;
    const float* k3;
    int act;
};

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Programmatic dependent launch.  Every kernel of the library is launched with programmatic
// stream serialization allowed and opens with pdl_wait(): nothing of the previous kernel in the
// stream is read or overwritten before that kernel has completed and its writes are visible.
// pdl_launch() then lets the next kernel's blocks be scheduled as soon as SM resources free up,
// so its launch latency overlaps this kernel's execution.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act == ACT_RELU6) return fminf(fmaxf(v, 0.f), 6.f);
    if (act == ACT_RELU) return fmaxf(v, 0.f);
    return v;
}
// 1 strictly inside the linear region, 0 at and beyond the kinks
__device__ __forceinline__ float act_mask(float pre, int act) {
    if (act == ACT_RELU6) return (pre > 0.f && pre < 6.f) ? 1.f : 0.f;
    if (act == ACT_RELU) return pre > 0.f ? 1.f : 0.f;
    return 1.f;
}

template <typename T> __device__ __forceinline__ float ld_val(const ValSrc& s, size_t idx, int c) {
    float z = to_f<T>(reinterpret_cast<const T*>(s.p)[idx]);
    if (s.scale) z = fmaf(z, __ldg(s.scale + c), __ldg(s.shift + c));
    return apply_act(z, s.act);
}

template <typename T> __device__ __forceinline__ float ld_grad(const GradSrc& s, size_t idx, int c) {
    float d = to_f<T>(reinterpret_cast<const T*>(s.dy)[idx]);
    if (s.act == ACT_NONE && s.k1 == nullptr) return d;
    float z = to_f<T>(reinterpret_cast<const T*>(s.z)[idx]);
    float pre = s.scale ? fmaf(z, __ldg(s.scale + c), __ldg(s.shift + c)) : z;
    d *= act_mask(pre, s.act);
    if (s.k1) d = fmaf(__ldg(s.k1 + c), d, fmaf(__ldg(s.k3 + c), z, __ldg(s.k2 + c)));
    return d;
}

// ---- 16-byte vectors of the storage type -------------------------------------------------
template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    float4 raw;
    __device__ __forceinline__ void load(const void* p, size_t vec_idx) { raw = reinterpret_cast<const float4*>(p)[vec_idx]; }
    __device__ __forceinline__ void store(void* p, size_t vec_idx) const { reinterpret_cast<float4*>(p)[vec_idx] = raw; }
    __device__ __forceinline__ void unpack(float* f) const { f[0] = raw.x; f[1] = raw.y; f[2] = raw.z; f[3] = raw.w; }
    __device__ __forceinline__ void pack(const float* f) { raw = make_float4(f[0], f[1], f[2], f[3]); }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    uint4 raw;
    __device__ __forceinline__ void load(const void* p, size_t vec_idx) { raw = reinterpret_cast<const uint4*>(p)[vec_idx]; }
    __device__ __forceinline__ void store(void* p, size_t vec_idx) const { reinterpret_cast<uint4*>(p)[vec_idx] = raw; }
    __device__ __forceinline__ void unpack(float* f) const {
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ __forceinline__ void pack(const float* f) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        raw = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// Vector forms of ld_val / ld_grad: N consecutive channels starting at channel c0 of element
// vector `vec_idx` (index in units of vectors).
// The transforms on vectors already in registers (so that a kernel can issue the loads of several vectors before it
// transforms any of them).
template <typename T> __device__ __forceinline__ void val_from_raw(const ValSrc& s, const Vec<T>& v, int c0, float* out) {
    v.unpack(out);
    if (s.scale) {
#pragma unroll
        for (int i = 0; i < Vec<T>::N; ++i) out[i] = fmaf(out[i], __ldg(s.scale + c0 + i), __ldg(s.shift + c0 + i));
    }
    if (s.act != ACT_NONE) {
#pragma unroll
        for (int i = 0; i < Vec<T>::N; ++i) out[i] = apply_act(out[i], s.act);
    }
}
__host__ __device__ __forceinline__ bool grad_needs_z(const GradSrc& s) { return s.act != ACT_NONE || s.k1 != nullptr; }
template <typename T> __device__ __forceinline__ void grad_from_raw(const GradSrc& s, const Vec<T>& dy, const Vec<T>& zv, int c0, float* out) {
    dy.unpack(out);
    if (!grad_needs_z(s)) return;
    float z[Vec<T>::N];
    zv.unpack(z);
#pragma unroll
    for (int i = 0; i < Vec<T>::N; ++i) {
        float pre = s.scale ? fmaf(z[i], __ldg(s.scale + c0 + i), __ldg(s.shift + c0 + i)) : z[i];
        float d = out[i] * act_mask(pre, s.act);
        if (s.k1) d = fmaf(__ldg(s.k1 + c0 + i), d, fmaf(__ldg(s.k3 + c0 + i), z[i], __ldg(s.k2 + c0 + i)));
        out[i] = d;
    }
}

template <typename T> __device__ __forceinline__ void ld_val_vec(const ValSrc& s, size_t vec_idx, int c0, float* out) {
    Vec<T> v;
    v.load(s.p, vec_idx);
    val_from_raw<T>(s, v, c0, out);
}

template <typename T> __device__ __forceinline__ void ld_grad_vec(const GradSrc& s, size_t vec_idx, int c0, float* out) {
    Vec<T> v, z;
    v.load(s.dy, vec_idx);
    z.raw = v.raw;
    if (grad_needs_z(s)) z.load(s.z, vec_idx);
    grad_from_raw<T>(s, v, z, c0, out);
}

// Width-generic access: V == Vec<T>::N uses 16-byte vectors, V == 1 scalars (channel counts that
// are not a multiple of the vector width).  `e` is the element index of the first channel.
template <typename T, int V> __device__ __forceinline__ void ld_raw_w(const void* p, size_t e, float* out) {
    if (V == 1) {
        out[0] = to_f<T>(reinterpret_cast<const T*>(p)[e]);
    } else {
        Vec<T> v;
        v.load(p, e / V);
        v.unpack(out);
    }
}
template <typename T, int V> __device__ __forceinline__ void st_raw_w(void* p, size_t e, const float* in) {
    if (V == 1) {
        reinterpret_cast<T*>(p)[e] = from_f<T>(in[0]);
    } else {
        Vec<T> v;
        v.pack(in);
        v.store(p, e / V);
    }
}
template <typename T, int V> __device__ __forceinline__ void ld_val_w(const ValSrc& s, size_t e, int c0, float* out) {
    if (V == 1) out[0] = ld_val<T>(s, e, c0);
    else ld_val_vec<T>(s, e / V, c0, out);
}
template <typename T, int V> __device__ __forceinline__ void ld_grad_w(const GradSrc& s, size_t e, int c0, float* out) {
    if (V == 1) out[0] = ld_grad<T>(s, e, c0);
    else ld_grad_vec<T>(s, e / V, c0, out);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace ast
