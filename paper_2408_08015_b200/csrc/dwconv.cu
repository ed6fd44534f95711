// Depthwise 3x3 convolution, NHWC, 16-byte channel vectors: forward, backward-data and
// backward-weight.  All three are bandwidth-bound; the producer's BatchNorm+activation
// (forward) and the BatchNorm-backward transform of the incoming gradient (backward) are
// applied while loading, so no normalised tensor is ever written.
#include "kernels.h"

namespace ast {
namespace {

// One thread per (pixel, channel vector).  Consecutive threads take consecutive channel
// vectors of a pixel, then the next pixel of the row: loads are fully coalesced and the 3x3
// neighbourhood is shared through L1.
template <typename T> __global__ void __launch_bounds__(256) dw_fwd_kernel(ConvGeom g, ValSrc x, const float* __restrict__ w9c, T* __restrict__ z) {
    constexpr int V = Vec<T>::N;
    const int cv = g.ci / V;
    size_t total = (size_t)g.n * g.ho * g.wo * cv;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    int j = (int)(i % cv);
    size_t p = i / cv;
    int wo = (int)(p % g.wo);
    size_t t = p / g.wo;
    int ho = (int)(t % g.ho), n = (int)(t / g.ho);
    int c0 = j * V;
    float acc[V];
#pragma unroll
    for (int q = 0; q < V; ++q) acc[q] = 0.f;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        int hi = ho * g.stride - 1 + r;
        if (hi < 0 || hi >= g.hi) continue;
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            int wi = wo * g.stride - 1 + s;
            if (wi < 0 || wi >= g.wi) continue;
            float xv[V];
            ld_val_vec<T>(x, ((size_t)(n * g.hi + hi) * g.wi + wi) * cv + j, c0, xv);
            const float* wp = w9c + (r * 3 + s) * g.ci + c0;
#pragma unroll
            for (int q = 0; q < V; ++q) acc[q] = fmaf(xv[q], __ldg(wp + q), acc[q]);
        }
    }
    Vec<T> o;
    o.pack(acc);
    o.store(z, i);
}

template <typename T>
__global__ void __launch_bounds__(256) dw_bwd_data_kernel(ConvGeom g, GradSrc dz, const float* __restrict__ w9c, const T* addend, T* dx) {
    constexpr int V = Vec<T>::N;
    const int cv = g.ci / V;
    size_t total = (size_t)g.n * g.hi * g.wi * cv;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    int j = (int)(i % cv);
    size_t p = i / cv;
    int wi = (int)(p % g.wi);
    size_t t = p / g.wi;
    int hi = (int)(t % g.hi), n = (int)(t / g.hi);
    int c0 = j * V;
    float acc[V];
    if (addend) {
        Vec<T> a;
        a.load(addend, i);
        a.unpack(acc);
    } else {
#pragma unroll
        for (int q = 0; q < V; ++q) acc[q] = 0.f;
    }
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        int a = hi + 1 - r;
        if (a < 0 || (g.stride == 2 && (a & 1))) continue;
        int ho = a / g.stride;
        if (ho >= g.ho) continue;
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            int b = wi + 1 - s;
            if (b < 0 || (g.stride == 2 && (b & 1))) continue;
            int wo = b / g.stride;
            if (wo >= g.wo) continue;
            float dv[V];
            ld_grad_vec<T>(dz, ((size_t)(n * g.ho + ho) * g.wo + wo) * cv + j, c0, dv);
            const float* wp = w9c + (r * 3 + s) * g.ci + c0;
#pragma unroll
            for (int q = 0; q < V; ++q) acc[q] = fmaf(dv[q], __ldg(wp + q), acc[q]);
        }
    }
    Vec<T> o;
    o.pack(acc);
    o.store(dx, i);
}

// Weight gradient: per channel, nine sums over all output pixels.  A block owns `cw` channel
// vectors and a contiguous range of output pixels; a thread keeps its 9*V partial sums in
// registers, rows of the block are combined through shared memory, blocks through a partials
// array summed in fixed order by a second kernel (deterministic, no float atomics).
template <typename T>
__global__ void __launch_bounds__(256) dw_bwd_weight_kernel(ConvGeom g, GradSrc dz, ValSrc x, int cw, int rows, size_t pix_per_block,
                                                            float* __restrict__ partial) {
    constexpr int V = Vec<T>::N;
    extern __shared__ float red[];      // [rows][cw*V] per tap, reused tap by tap
    const int cv = g.ci / V;
    const int jl = threadIdx.x % cw, row = threadIdx.x / cw;
    const int j = blockIdx.x * cw + jl;
    const bool active = row < rows && j < cv;
    const int c0 = j * V;
    size_t P = (size_t)g.n * g.ho * g.wo;
    size_t pbeg = (size_t)blockIdx.y * pix_per_block, pend = min(P, pbeg + pix_per_block);
    float acc[9][V];
#pragma unroll
    for (int t = 0; t < 9; ++t)
#pragma unroll
        for (int q = 0; q < V; ++q) acc[t][q] = 0.f;
    if (active) {
        for (size_t p = pbeg + row; p < pend; p += rows) {
            int wo = (int)(p % g.wo);
            size_t t2 = p / g.wo;
            int ho = (int)(t2 % g.ho), n = (int)(t2 / g.ho);
            float dv[V];
            ld_grad_vec<T>(dz, p * cv + j, c0, dv);
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                int hi = ho * g.stride - 1 + r;
                if (hi < 0 || hi >= g.hi) continue;
#pragma unroll
                for (int s = 0; s < 3; ++s) {
                    int wi = wo * g.stride - 1 + s;
                    if (wi < 0 || wi >= g.wi) continue;
                    float xv[V];
                    ld_val_vec<T>(x, ((size_t)(n * g.hi + hi) * g.wi + wi) * cv + j, c0, xv);
#pragma unroll
                    for (int q = 0; q < V; ++q) acc[r * 3 + s][q] = fmaf(dv[q], xv[q], acc[r * 3 + s][q]);
                }
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
            int c = blockIdx.x * width + e;
            if (c < g.ci) {
                float s = 0.f;
                for (int r2 = 0; r2 < rows; ++r2) s += red[r2 * width + e];
                partial[((size_t)blockIdx.y * 9 + t) * g.ci + c] = s;
            }
        }
        __syncthreads();
    }
}

// gw[c][t] = sum_b partial[b][t][c]
__global__ void dw_bwd_weight_finish(const float* __restrict__ partial, int blocks, int c_total, float* __restrict__ gw) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 9 * c_total) return;
    int t = i / c_total, c = i % c_total;
    float s = 0.f;
    for (int b = 0; b < blocks; ++b) s += partial[((size_t)b * 9 + t) * c_total + c];
    gw[c * 9 + t] = s;
}

}  // namespace

static double esz(int dtype) { return dtype == 0 ? 4.0 : 2.0; }
static double grad_src_bytes(const GradSrc& d, double elems, int dtype) { return elems * esz(dtype) * ((d.act != ACT_NONE || d.k1) ? 2.0 : 1.0); }

void dw_fwd(int dtype, const ConvGeom& g, const ValSrc& x, const float* w9c, void* z, cudaStream_t st) {
    double in_e = (double)g.n * g.hi * g.wi * g.ci, out_e = (double)g.n * g.ho * g.wo * g.ci;
    LaunchScope ls(K_DW_FWD, (in_e + out_e) * esz(dtype) + 36.0 * g.ci, 18.0 * out_e, st);
    if (dtype == 0) {
        size_t total = (size_t)g.n * g.ho * g.wo * (g.ci / 4);
        dw_fwd_kernel<float><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(g, x, w9c, (float*)z);
    } else {
        size_t total = (size_t)g.n * g.ho * g.wo * (g.ci / 8);
        dw_fwd_kernel<__nv_bfloat16><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(g, x, w9c, (__nv_bfloat16*)z);
    }
}

void dw_bwd_data(int dtype, const ConvGeom& g, const GradSrc& dz, const float* w9c, const void* addend, void* dx, cudaStream_t st) {
    double in_e = (double)g.n * g.hi * g.wi * g.ci, out_e = (double)g.n * g.ho * g.wo * g.ci;
    LaunchScope ls(K_DW_BWD_DATA, grad_src_bytes(dz, out_e, dtype) + in_e * esz(dtype) * (addend ? 2.0 : 1.0) + 36.0 * g.ci, 18.0 * out_e, st);
    if (dtype == 0) {
        size_t total = (size_t)g.n * g.hi * g.wi * (g.ci / 4);
        dw_bwd_data_kernel<float><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(g, dz, w9c, (const float*)addend, (float*)dx);
    } else {
        size_t total = (size_t)g.n * g.hi * g.wi * (g.ci / 8);
        dw_bwd_data_kernel<__nv_bfloat16><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(g, dz, w9c, (const __nv_bfloat16*)addend, (__nv_bfloat16*)dx);
    }
}

void dw_bwd_weight(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw,
                   cudaStream_t st) {
    const int V = dtype == 0 ? 4 : 8;
    const int cv = g.ci / V;
    int cw = cv < 32 ? cv : 32;
    int rows = 256 / cw;
    size_t P = (size_t)g.n * g.ho * g.wo;
    int gx = (cv + cw - 1) / cw;
    size_t by = (4 * 148 + gx - 1) / gx;
    size_t max_by = (P + (size_t)rows * 4 - 1) / ((size_t)rows * 4);
    if (by > max_by) by = max_by;
    size_t cap = scratch_floats / ((size_t)9 * g.ci);
    if (by > cap) by = cap;
    if (by < 1) by = 1;
    size_t ppb = (P + by - 1) / by;
    by = (P + ppb - 1) / ppb;
    size_t smem = (size_t)rows * cw * V * sizeof(float);
    dim3 grid(gx, (unsigned)by);
    double in_e = (double)g.n * g.hi * g.wi * g.ci, out_e = (double)P * g.ci;
    {
        LaunchScope ls(K_DW_BWD_WEIGHT, grad_src_bytes(dz, out_e, dtype) + in_e * esz(dtype) + 36.0 * g.ci * by, 18.0 * out_e, st);
        if (dtype == 0)
            dw_bwd_weight_kernel<float><<<grid, 256, smem, st>>>(g, dz, x, cw, rows, ppb, scratch);
        else
            dw_bwd_weight_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>(g, dz, x, cw, rows, ppb, scratch);
    }
    LaunchScope ls(K_DW_BWD_WEIGHT_FINISH, 36.0 * g.ci * (by + 1), 9.0 * g.ci * by, st);
    dw_bwd_weight_finish<<<(9 * g.ci + 255) / 256, 256, 0, st>>>(scratch, (int)by, g.ci, gw);
}

}  // namespace ast
