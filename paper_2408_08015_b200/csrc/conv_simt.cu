// Dense convolution (any k, stride, pad) as an implicit GEMM on plain FFMA tiles.
// This is the float32 path (TF32/bf16 tensor tiles are too coarse for a 1e-4 bound) and the
// general fallback for shapes the tensor-core kernels do not take.
//
//   forward      C[p][ko] = sum_kk A[p][kk] * W[ko][kk]      kk = (r,s,c),  A gathered from x
//   bwd-data     C[q][c]  = sum_kk D[q][kk] * Wt[c][kk]      kk = (r,s,ko), D gathered from dz
//   bwd-weight   C[ko][j] = sum_p  dz[p][ko] * A[p][j]       j  = (r,s,c),  reduction over pixels, split
#include "kernels.h"

namespace ast {

namespace {

constexpr int BM = 64, BN = 64, BK = 16, NT = 256;
enum { MODE_FWD = 0, MODE_BWD_DATA = 1, MODE_BWD_WEIGHT = 2 };

struct IgemmArgs {
    ConvGeom g;
    ValSrc x;
    GradSrc dz;
    const float* w;       // FWD: w[ko][r][s][c]; BWD_DATA: wt[c][r][s][ko]
    const float* bias;
    const void* addend;
    void* out;
    float* partial;
    int M, N, K;
    int k_per_split;
};

// input pixel of x feeding output (ho,wo) through tap (r,s); returns false if in the padding
__device__ __forceinline__ bool tap_in(const ConvGeom& g, int ho, int wo, int r, int s, int& hi, int& wi) {
    hi = ho * g.stride - g.pad + r;
    wi = wo * g.stride - g.pad + s;
    return hi >= 0 && hi < g.hi && wi >= 0 && wi < g.wi;
}
// output pixel of dz that input (hi,wi) feeds through tap (r,s)
__device__ __forceinline__ bool tap_out(const ConvGeom& g, int hi, int wi, int r, int s, int& ho, int& wo) {
    int a = hi + g.pad - r, b = wi + g.pad - s;
    if (a < 0 || b < 0) return false;
    if (g.stride > 1 && ((a % g.stride) | (b % g.stride))) return false;
    ho = a / g.stride;
    wo = b / g.stride;
    return ho < g.ho && wo < g.wo;
}

// Operands of a dense contraction are bf16 values in bfloat16 mode (the tensor-core input
// format), whichever kernel executes the layer; accumulation is float32.
template <typename T> __device__ __forceinline__ float operand(float v) { return v; }
template <> __device__ __forceinline__ float operand<__nv_bfloat16>(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

template <typename T, int MODE> __global__ void __launch_bounds__(NT) igemm_kernel(const IgemmArgs a) {
    pdl_wait();
    pdl_launch();
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const ConvGeom& g = a.g;
    const int tid = threadIdx.x;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int tx = tid % 16, ty = tid / 16;
    float acc[4][4] = {};

    int kbeg = 0, kend = a.K;
    if (MODE == MODE_BWD_WEIGHT) {
        kbeg = blockIdx.z * a.k_per_split;
        kend = min(a.K, kbeg + a.k_per_split);
    }

    // ---- per-thread fixed coordinates of the elements it stages ----
    // FWD / BWD_DATA: A row = tid/4 (a pixel), 4 consecutive kk; B row = tid/4 (a channel), 4 consecutive kk.
    // BWD_WEIGHT: kk = tid/16 (a pixel), 4 consecutive rows of A (ko) and of B (j).
    int pa_n = 0, pa_h = 0, pa_w = 0;
    bool row_ok = false;
    int jb_r[4], jb_s[4], jb_c[4];
    if (MODE != MODE_BWD_WEIGHT) {
        int m = m0 + tid / 4;
        row_ok = m < a.M;
        int hh = (MODE == MODE_FWD) ? g.ho : g.hi, ww = (MODE == MODE_FWD) ? g.wo : g.wi;
        if (row_ok) {
            pa_w = m % ww;
            int t = m / ww;
            pa_h = t % hh;
            pa_n = t / hh;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int col = n0 + (tid % 16) * 4 + j;
            jb_c[j] = col % g.ci;
            int rs = col / g.ci;
            jb_s[j] = rs % g.k;
            jb_r[j] = rs / g.k;
            if (col >= a.N) jb_r[j] = -1;
        }
    }

    for (int k0 = kbeg; k0 < kend; k0 += BK) {
        if (MODE == MODE_FWD || MODE == MODE_BWD_DATA) {
            const int ch = (MODE == MODE_FWD) ? g.ci : g.co;   // channels of the gathered tensor
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int kl = (tid % 4) * 4 + j, kk = k0 + kl;
                float va = 0.f, vb = 0.f;
                if (kk < kend) {
                    int c = kk % ch, rs = kk / ch;
                    int s = rs % g.k, r = rs / g.k;
                    if (row_ok) {
                        int h2, w2;
                        if (MODE == MODE_FWD) {
                            if (tap_in(g, pa_h, pa_w, r, s, h2, w2))
                                va = ld_val<T>(a.x, ((size_t)(pa_n * g.hi + h2) * g.wi + w2) * g.ci + c, c);
                        } else {
                            if (tap_out(g, pa_h, pa_w, r, s, h2, w2))
                                va = ld_grad<T>(a.dz, ((size_t)(pa_n * g.ho + h2) * g.wo + w2) * g.co + c, c);
                        }
                    }
                    int nb = n0 + tid / 4;
                    if (nb < a.N) vb = __ldg(a.w + (size_t)nb * a.K + kk);
                }
                As[kl][tid / 4] = operand<T>(va);
                Bs[kl][tid / 4] = operand<T>(vb);
            }
        } else {
            int kl = tid / 16, p = k0 + kl;
            bool p_ok = p < kend;
            int pn = 0, ph = 0, pw = 0;
            if (p_ok) {
                pw = p % g.wo;
                int t = p / g.wo;
                ph = t % g.ho;
                pn = t / g.ho;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int ml = (tid % 16) * 4 + j, ko = m0 + ml;
                float va = 0.f, vb = 0.f;
                if (p_ok) {
                    if (ko < a.M) va = ld_grad<T>(a.dz, (size_t)p * g.co + ko, ko);
                    int h2, w2;
                    if (jb_r[j] >= 0 && tap_in(g, ph, pw, jb_r[j], jb_s[j], h2, w2))
                        vb = ld_val<T>(a.x, ((size_t)(pn * g.hi + h2) * g.wi + w2) * g.ci + jb_c[j], jb_c[j]);
                }
                As[kl][ml] = operand<T>(va);
                Bs[kl][ml] = operand<T>(vb);
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float ar[4] = {av.x, av.y, av.z, av.w}, br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
        }
        __syncthreads();
    }

    // ---- epilogue ----
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty * 4 + i;
        if (m >= a.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int n = n0 + tx * 4 + j;
            if (n >= a.N) continue;
            size_t idx = (size_t)m * a.N + n;
            float v = acc[i][j];
            if (MODE == MODE_BWD_WEIGHT) {
                a.partial[(size_t)blockIdx.z * a.M * a.N + idx] = v;
            } else {
                if (MODE == MODE_FWD && a.bias) v += __ldg(a.bias + n);
                if (MODE == MODE_BWD_DATA && a.addend) v += to_f<T>(reinterpret_cast<const T*>(a.addend)[idx]);
                reinterpret_cast<T*>(a.out)[idx] = from_f<T>(v);
            }
        }
    }
}

__global__ void reduce_splits_kernel(const float* __restrict__ partial, int splits, size_t n, float* __restrict__ out) {
    pdl_wait();
    pdl_launch();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.f;
    for (int k0 = 0; k0 < splits; k0 += 8) {      // eight loads in flight, additions in index order
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = (k0 + u < splits) ? partial[(size_t)(k0 + u) * n + i] : 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) s += v[u];
    }
    out[i] = s;
}

// ---- small-c_in dense convs (the 3-channel stem) as an explicit im2col + pointwise tensor-core GEMM ----
// col[p][kk] = x value feeding output pixel p through tap kk = (r, s, c) (the weight layout's order), zero in the
// padding and for kk >= K; rows are Kp bf16 values (Kp a multiple of 8, at most 64).  One thread writes one pixel's
// row; the decomposition of kk (tap row, tap column, channel, offset from the pixel's first input element) comes from
// a table in shared memory, so that the per-element work is a lookup, two bit tests and a load.
__global__ void __launch_bounds__(256) im2col_kernel(ConvGeom g, ValSrc x, int K, int Kp, __nv_bfloat16* __restrict__ col, size_t pixels) {
    pdl_launch();
    __shared__ int t_off[64];
    __shared__ unsigned char t_r[64], t_s[64], t_c[64];
    for (int kk = threadIdx.x; kk < Kp; kk += blockDim.x) {
        int c = 0, r = 31, s2 = 31, off = 0;         // kk >= K: a tap position no mask has
        if (kk < K) {
            c = kk % g.ci;
            const int rs = kk / g.ci;
            s2 = rs % g.k;
            r = rs / g.k;
            off = (r * g.wi + s2) * g.ci + c;
        }
        t_off[kk] = off; t_r[kk] = (unsigned char)r; t_s[kk] = (unsigned char)s2; t_c[kk] = (unsigned char)c;
    }
    __syncthreads();
    pdl_wait();
    const size_t p = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= pixels) return;
    const int wo = (int)(p % g.wo);
    const size_t t = p / g.wo;
    const int ho = (int)(t % g.ho), n = (int)(t / g.ho);
    const int h0 = ho * g.stride - g.pad, w0 = wo * g.stride - g.pad;
    unsigned rmask = 0, smask = 0;                   // taps whose input row / column lies inside the image
    for (int q = 0; q < g.k; ++q) {
        rmask |= (h0 + q >= 0 && h0 + q < g.hi) ? (1u << q) : 0u;
        smask |= (w0 + q >= 0 && w0 + q < g.wi) ? (1u << q) : 0u;
    }
    const long long base = ((long long)(n * g.hi + h0) * g.wi + w0) * g.ci;
    uint4* dst = reinterpret_cast<uint4*>(col + p * (size_t)Kp);
    for (int j = 0; j < (Kp >> 3); ++j) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float v2[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int kk = (j << 3) + 2 * q + e;
                const bool ok = ((rmask >> t_r[kk]) & (smask >> t_s[kk]) & 1u) != 0;
                v2[e] = ok ? ld_val<__nv_bfloat16>(x, (size_t)(base + t_off[kk]), t_c[kk]) : 0.f;
            }
            __nv_bfloat162 h = __floats2bfloat162_rn(v2[0], v2[1]);
            w[q] = *reinterpret_cast<uint32_t*>(&h);
        }
        dst[j] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// wpad[ko][kk] = bf16(w[ko][kk]) for kk < K, zero up to Kp
__global__ void pad_weights_kernel(const float* __restrict__ w, int co, int K, int Kp, __nv_bfloat16* __restrict__ wpad) {
    pdl_wait();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < co * Kp) {
        const int ko = i / Kp, kk = i - ko * Kp;
        wpad[i] = __float2bfloat16_rn(kk < K ? w[(size_t)ko * K + kk] : 0.f);
    }
    // no early release of the dependents: other kernels stage these weights before their dependency wait (see refresh_kernel)
}

// gw[ko][kk] = gpad[ko][kk], kk < K
__global__ void unpad_grad_kernel(const float* __restrict__ gpad, int co, int K, int Kp, float* __restrict__ gw) {
    pdl_wait();
    pdl_launch();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= co * K) return;
    const int ko = i / K, kk = i - ko * K;
    gw[i] = gpad[(size_t)ko * Kp + kk];
}

template <int MODE> void launch(int dtype, const IgemmArgs& a, dim3 grid, int kind, double bytes, cudaStream_t st) {
    LaunchScope ls(kind, bytes, 2.0 * a.M * a.N * a.K, st);
    if (dtype == 0)
        launch_pdl(igemm_kernel<float, MODE>, grid, NT, 0, st, a);
    else
        launch_pdl(igemm_kernel<__nv_bfloat16, MODE>, grid, NT, 0, st, a);
}

double esz(int dtype) { return dtype == 0 ? 4.0 : 2.0; }
// bytes read to form dz on load: dy always, z when a mask or BatchNorm backward is applied
double grad_src_bytes(const GradSrc& d, double elems, int dtype) { return elems * esz(dtype) * ((d.act != ACT_NONE || d.k1) ? 2.0 : 1.0); }

}  // namespace

void conv_fwd(int dtype, const ConvGeom& g, const ValSrc& x, const float* w, const float* bias, void* z, cudaStream_t st) {
    IgemmArgs a{};
    a.g = g; a.x = x; a.w = w; a.bias = bias; a.out = z;
    a.M = g.n * g.ho * g.wo; a.N = g.co; a.K = g.k * g.k * g.ci;
    double bytes = ((double)g.n * g.hi * g.wi * g.ci + (double)a.M * a.N) * esz(dtype) + 4.0 * a.N * a.K;
    launch<MODE_FWD>(dtype, a, dim3((a.M + BM - 1) / BM, (a.N + BN - 1) / BN, 1), K_CONV_FWD, bytes, st);
}

void conv_bwd_data(int dtype, const ConvGeom& g, const GradSrc& dz, const float* wt, const void* addend, void* dx, cudaStream_t st) {
    IgemmArgs a{};
    a.g = g; a.dz = dz; a.w = wt; a.addend = addend; a.out = dx;
    a.M = g.n * g.hi * g.wi; a.N = g.ci; a.K = g.k * g.k * g.co;
    double bytes = grad_src_bytes(dz, (double)g.n * g.ho * g.wo * g.co, dtype) + (double)a.M * a.N * esz(dtype) * (addend ? 2.0 : 1.0) +
                   4.0 * a.N * a.K;
    launch<MODE_BWD_DATA>(dtype, a, dim3((a.M + BM - 1) / BM, (a.N + BN - 1) / BN, 1), K_CONV_BWD_DATA, bytes, st);
}

void conv_bwd_weight(int dtype, const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats,
                     float* gw, cudaStream_t st) {
    IgemmArgs a{};
    a.g = g; a.dz = dz; a.x = x; a.partial = scratch;
    a.M = g.co; a.N = g.k * g.k * g.ci; a.K = g.n * g.ho * g.wo;
    int tiles = ((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN);
    size_t out_elems = (size_t)a.M * a.N;
    int splits = (4 * sm_count() + tiles - 1) / tiles;
    int max_by_k = (a.K + 4 * BK - 1) / (4 * BK);
    if (splits > max_by_k) splits = max_by_k;
    size_t cap = scratch_floats / out_elems;
    if ((size_t)splits > cap) splits = (int)cap;
    if (splits < 1) splits = 1;
    int kps = (a.K + splits - 1) / splits;
    kps = (kps + BK - 1) / BK * BK;
    splits = (a.K + kps - 1) / kps;
    a.k_per_split = kps;
    double bytes = grad_src_bytes(dz, (double)a.K * g.co, dtype) + (double)g.n * g.hi * g.wi * g.ci * esz(dtype) + 4.0 * out_elems * splits;
    launch<MODE_BWD_WEIGHT>(dtype, a, dim3((a.M + BM - 1) / BM, (a.N + BN - 1) / BN, splits), K_CONV_BWD_WEIGHT, bytes, st);
    LaunchScope ls(K_REDUCE_SPLITS, 4.0 * out_elems * (splits + 1), (double)out_elems * splits, st);
    launch_pdl(reduce_splits_kernel, (unsigned)((out_elems + 255) / 256), 256, 0, st, scratch, splits, out_elems, gw);
}

void conv_im2col(const ConvGeom& g, const ValSrc& x, int Kp, void* col, cudaStream_t st) {
    const int K = g.k * g.k * g.ci;
    const size_t pixels = (size_t)g.n * g.ho * g.wo;
    LaunchScope ls(K_IM2COL, 2.0 * ((double)g.n * g.hi * g.wi * g.ci + (double)pixels * Kp), 0.0, st);
    launch_pdl(im2col_kernel, (unsigned)((pixels + 255) / 256), 256, 0, st, g, x, K, Kp, (__nv_bfloat16*)col, pixels);
}

void conv_pad_weights(const float* w, int co, int K, int Kp, __nv_bfloat16* wpad, cudaStream_t st) {
    LaunchScope ls(K_COL_AUX, 4.0 * co * K + 2.0 * co * Kp, 0.0, st);
    launch_pdl(pad_weights_kernel, (co * Kp + 255) / 256, 256, 0, st, w, co, K, Kp, wpad);
}

void conv_unpad_grad(const float* gpad, int co, int K, int Kp, float* gw, cudaStream_t st) {
    LaunchScope ls(K_COL_AUX, 8.0 * co * K, 0.0, st);
    launch_pdl(unpad_grad_kernel, (co * K + 255) / 256, 256, 0, st, gpad, co, K, Kp, gw);
}

}  // namespace ast
