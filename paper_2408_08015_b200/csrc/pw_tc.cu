// Pointwise (1x1) convolution on the 5th-generation tensor cores: forward and backward-data.
//
//   forward    Z[p][n]  = sum_c A[p][c] * W[n][c],    A[p][c] = act(x[p][c]*scale[c] + shift[c])
//   bwd-data   dX[p][c] = sum_k D[p][k] * Wt[c][k],   D = BatchNorm/activation backward of dy, formed on load
//
// Both are one GEMM  C[128 pixels x NT] += A[128 x K] * B[NT x K]^T  per CTA with bf16 operands
// and float32 accumulation in tensor memory (tcgen05.mma, cta_group::1, M = 128).  The A operand
// cannot come straight from global memory by a bulk copy because the producer's BatchNorm and
// activation (or, backward, the BatchNorm-backward transform) are applied on the way: all
// threads load 16-byte channel vectors, transform them in registers and store bf16 into shared
// memory in the K-major 128-byte-swizzled layout the MMA reads.  These layers are HBM-bound
// (K and N are small), so a CTA holds one 128-pixel tile and several CTAs per SM overlap
// their load, MMA and store phases.  Every wait is bounded and reports through an error word.
#include <cuda_bf16.h>

#include "kernels.h"

namespace ast {
namespace {

constexpr int TM = 128;            // pixels per CTA (UMMA M)
constexpr int NTHREADS = 256;
constexpr int KB = 64;             // bf16 elements per 128-byte swizzle row
constexpr uint32_t WAIT_LIMIT = 1u << 22;

struct PwArgs {
    ValSrc x;              // forward operand
    GradSrc dz;            // backward operand
    const __nv_bfloat16* w;   // [N][K], K contiguous
    const float* bias;     // forward only, may be null
    const void* addend;    // backward only, may be null ([P][N])
    __nv_bfloat16* out;    // [P][N]
    int* err;              // device error word: set to 1 if a wait ran out
    int P, K, N;           // output pixels, reduction length, output channels
    int NT;                // output channels per CTA (multiple of 16, <= 256)
    int KC;                // reduction elements staged at once (multiple of 64)
    int tmem_cols;         // power of two >= 32, >= NT
    // spatial subsampling of the forward operand (1x1 conv with stride): output pixel -> input pixel
    int stride, ho, wo, hi, wi;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t mbar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mbar) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t mbar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(mbar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within WAIT_LIMIT polls.
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity) {
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(mbar, parity)) return true;
        if (i > 64) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows are 128 bytes apart,
// groups of 8 rows 1024 bytes apart (stride-dimension offset); 16-byte chunk j of row r sits at
// chunk position j ^ (r & 7).  The leading-dimension offset is not used by swizzled K-major
// layouts.  Bits: [0,14) address>>4, [16,30) LBO>>4, [32,46) SBO>>4, [46,48) version 1,
// [61,64) layout 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor, kind::f16: D = f32 (bit 4), A = B = bf16 (bits 7, 10), both K-major,
// N>>3 at bit 17, M>>4 at bit 24.
__device__ __forceinline__ uint32_t make_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
}

// byte offset of 16-byte chunk `j` (8 bf16) of row `r` inside an operand staged as 64-element
// K blocks of `rows` rows each
__device__ __forceinline__ uint32_t tile_off(int r, int j, int rows) {
    int kb = j >> 3, jj = j & 7;
    return (uint32_t)kb * (uint32_t)rows * 128u + (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u + (uint32_t)((jj ^ (r & 7)) << 4);
}

__device__ __forceinline__ uint4 pack8(const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

template <bool BWD> __global__ void __launch_bounds__(NTHREADS) pw_tc_kernel(const PwArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t mbar_store;
    __shared__ uint32_t tmem_slot;
    __shared__ int failed;
    // 1024-byte aligned operand area (the swizzle pattern is a function of the address bits)
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int NT = a.NT;
    uint8_t* sA = base;
    uint8_t* sB = base + (size_t)(a.KC / KB) * TM * 128;
    const uint32_t mbar = smem_u32(&mbar_store);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int p0 = blockIdx.x * TM;
    const int n0 = blockIdx.y * NT;

    if (tid == 0) {
        mbar_init(mbar, 1);
        failed = 0;
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), (uint32_t)a.tmem_cols);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = tmem_slot;
    const uint32_t idesc = make_idesc(NT);

    uint32_t phase = 0;
    bool ok = true;
    for (int k0 = 0; k0 < a.K; k0 += a.KC) {
        const int kc = min(a.KC, a.K - k0);           // multiple of 8
        const int vpr = kc >> 3;                      // 16-byte vectors per row holding data
        const int vpr_pad = ((kc + 15) >> 4) << 1;    // rounded up to whole MMA k-steps
        // ---- stage A: [128 pixels][kc] ----
        for (int v = tid; v < TM * vpr_pad; v += NTHREADS) {
            int r = v / vpr_pad, j = v - r * vpr_pad;
            int p = p0 + r;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (p < a.P && j < vpr) {
                float f[8];
                int c0 = k0 + (j << 3);
                if (BWD) {
                    ld_grad_vec<__nv_bfloat16>(a.dz, ((size_t)p * a.K + c0) >> 3, c0, f);
                } else {
                    size_t pin = p;
                    if (a.stride > 1) {
                        int wo = p % a.wo, t = p / a.wo;
                        int ho = t % a.ho, n = t / a.ho;
                        pin = ((size_t)n * a.hi + (size_t)ho * a.stride) * a.wi + (size_t)wo * a.stride;
                    }
                    ld_val_vec<__nv_bfloat16>(a.x, (pin * a.K + c0) >> 3, c0, f);
                }
                q = pack8(f);
            }
            *reinterpret_cast<uint4*>(sA + tile_off(r, j, TM)) = q;
        }
        // ---- stage B: [NT channels][kc] of the bf16 weights ----
        for (int v = tid; v < NT * vpr_pad; v += NTHREADS) {
            int r = v / vpr_pad, j = v - r * vpr_pad;
            int n = n0 + r;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (n < a.N && j < vpr) q = __ldg(reinterpret_cast<const uint4*>(a.w + (size_t)n * a.K + k0) + j);
            *reinterpret_cast<uint4*>(sB + tile_off(r, j, NT)) = q;
        }
        fence_async_smem();
        __syncthreads();
        if (tid == 0) {
            fence_after_sync();
            const uint32_t a0 = smem_u32(sA), b0 = smem_u32(sB);
            const int steps = vpr_pad >> 1;           // 16 elements per MMA
            for (int s = 0; s < steps; ++s) {
                int kb = s >> 2, ks = s & 3;          // 64-element block, 32-byte step inside it
                uint64_t da = make_desc(a0 + (uint32_t)kb * TM * 128u + (uint32_t)ks * 32u);
                uint64_t db = make_desc(b0 + (uint32_t)kb * (uint32_t)NT * 128u + (uint32_t)ks * 32u);
                umma_bf16(tmem, da, db, idesc, (k0 > 0 || s > 0) ? 1u : 0u);
            }
            umma_commit(mbar);
        }
        // all threads wait until the MMAs have consumed shared memory / produced the accumulators
        ok = mbar_wait(mbar, phase);
        phase ^= 1;
        if (!__syncthreads_and(ok ? 1 : 0)) {   // uniform decision: every thread leaves the loop together
            if (tid == 0) failed = 1;
            break;
        }
    }
    fence_after_sync();
    __syncthreads();
    if (failed) {
        if (tid == 0) atomicExch(a.err, 1);
    } else {
        // ---- epilogue: warp w reads lane quarter (w & 3); column groups of 8 alternate between the two warp sets ----
        const int q = warp & 3, half = warp >> 2;
        const int row = q * 32 + lane, p = p0 + row;
        for (int g = half; g < (NT >> 3); g += 2) {
            float v[8];
            tmem_ld8(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g << 3), v);
            int n = n0 + (g << 3);
            if (p < a.P && n < a.N) {
                size_t e = (size_t)p * a.N + n;
                if (!BWD && a.bias) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] += __ldg(a.bias + n + i);
                }
                if (BWD && a.addend) {
                    float ad[8];
                    Vec<__nv_bfloat16> av;
                    av.load(a.addend, e >> 3);
                    av.unpack(ad);
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] += ad[i];
                }
                *reinterpret_cast<uint4*>(a.out + e) = pack8(v);
            }
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
}


// ---------------------------------------------------------------------------------------------
// Weight gradient of a pointwise conv:  gw[k][c] = sum_p dz[p][k] * x[p][c].
// D[128 x N] (rows = output channels k, columns = input channels c) accumulates in tensor memory
// over the CTA's pixel range; the reduction dimension is the pixel, so both operands are read
// exactly as they lie in global memory ([pixel][channel]) and staged MN-major: a stage holds 64
// pixels as rows of 128 bytes (64 channels) per channel panel, 8-row groups 1024 bytes apart
// (stride-dimension offset), panels 8192 bytes apart (leading-dimension offset), 16-byte chunks
// XOR-swizzled with the row index.  Two stage buffers: the MMAs of one stage run while the next
// is being loaded and transformed.  Rows/columns beyond the valid channels hold stale data and
// only feed accumulator rows/columns that are never read; pixel rows beyond the range are zeroed.
constexpr int WSTAGE = 64;                 // pixels per stage
constexpr int PANEL = WSTAGE * 128;        // bytes of one 64-channel panel of a stage

struct PwWArgs {
    GradSrc dz;
    ValSrc x;
    float* partial;        // [splits][CO][CI]
    int* err;
    int P, CO, CI;         // output pixels, output channels, input channels
    int pix_per_cta;       // multiple of WSTAGE
    int NT;                // input channels per CTA (multiple of 16, <= 256)
    int tmem_cols;
    int stride, ho, wo, hi, wi;
};

__device__ __forceinline__ uint64_t make_desc_mn(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(PANEL >> 4) << 16;     // leading-dimension offset: next 64-channel panel
    d |= (uint64_t)(1024 >> 4) << 32;      // stride-dimension offset: next group of 8 pixels
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

__global__ void __launch_bounds__(NTHREADS) pw_bwd_weight_tc_kernel(const PwWArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t mbar_store[2];
    __shared__ uint32_t tmem_slot;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * TM;                    // first output channel of this CTA
    const int n0 = blockIdx.z * a.NT;                  // first input channel
    const int ca = min(TM, a.CO - m0) >> 3;            // 16-byte chunks per pixel of the A operand
    const int cb = min(a.NT, a.CI - n0) >> 3;
    const int pa = (ca + 7) >> 3, pb = (cb + 7) >> 3;  // 64-channel panels
    const int nb_panels = (a.NT + 63) >> 6;
    const uint32_t buf_bytes = (uint32_t)(2 + nb_panels) * PANEL;
    const int pbeg = blockIdx.y * a.pix_per_cta, pend = min(a.P, pbeg + a.pix_per_cta);
    const uint32_t mbar0 = smem_u32(&mbar_store[0]), mbar1 = smem_u32(&mbar_store[1]);

    if (tid == 0) {
        mbar_init(mbar0, 1);
        mbar_init(mbar1, 1);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), (uint32_t)a.tmem_cols);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = tmem_slot;
    // D = f32, A = B = bf16, both MN-major (bits 15, 16)
    const uint32_t idesc = make_idesc(a.NT) | (1u << 15) | (1u << 16);

    uint32_t ph[2] = {0, 0};
    int issued[2] = {0, 0};
    bool ok = true, bad = false;       // `bad` is decided by a block-wide vote: uniform across threads
    int stage = 0;
    for (int ps = pbeg; ps < pend; ps += WSTAGE, ++stage) {
        const int b = stage & 1;
        uint8_t* sA = base + (size_t)b * buf_bytes;
        uint8_t* sB = sA + 2 * PANEL;
        if (issued[b]) {                               // the MMAs that read this buffer two stages ago
            ok = mbar_wait(b ? mbar1 : mbar0, ph[b]);
            ph[b] ^= 1;
        }
        if (!__syncthreads_and(ok ? 1 : 0)) {
            bad = true;
            break;
        }
        const int valid = min(WSTAGE, pend - ps);
        for (int v = tid; v < WSTAGE * ca; v += NTHREADS) {
            int kr = v / ca, j = v - kr * ca;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (kr < valid) {
                float f[8];
                int c0 = m0 + (j << 3);
                ld_grad_vec<__nv_bfloat16>(a.dz, ((size_t)(ps + kr) * a.CO + c0) >> 3, c0, f);
                q = pack8(f);
            }
            *reinterpret_cast<uint4*>(sA + (j >> 3) * PANEL + kr * 128 + (((j & 7) ^ (kr & 7)) << 4)) = q;
        }
        for (int v = tid; v < WSTAGE * cb; v += NTHREADS) {
            int kr = v / cb, j = v - kr * cb;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (kr < valid) {
                float f[8];
                int c0 = n0 + (j << 3);
                size_t pin = ps + kr;
                if (a.stride > 1) {
                    int p = ps + kr;
                    int wo = p % a.wo, t = p / a.wo;
                    int ho = t % a.ho, n = t / a.ho;
                    pin = ((size_t)n * a.hi + (size_t)ho * a.stride) * a.wi + (size_t)wo * a.stride;
                }
                ld_val_vec<__nv_bfloat16>(a.x, (pin * a.CI + c0) >> 3, c0, f);
                q = pack8(f);
            }
            *reinterpret_cast<uint4*>(sB + (j >> 3) * PANEL + kr * 128 + (((j & 7) ^ (kr & 7)) << 4)) = q;
        }
        fence_async_smem();
        __syncthreads();
        if (tid == 0) {
            fence_after_sync();
            const uint32_t a0 = smem_u32(sA), b0 = smem_u32(sB);
#pragma unroll
            for (int s = 0; s < WSTAGE / 16; ++s)      // 16 pixels = two 8-row groups per MMA
                umma_bf16(tmem, make_desc_mn(a0 + s * 2048), make_desc_mn(b0 + s * 2048), idesc, (stage > 0 || s > 0) ? 1u : 0u);
            umma_commit(b ? mbar1 : mbar0);
        }
        issued[b] = 1;
    }
    // drain: the last commit covers every earlier MMA of the issuing thread
    if (!bad && stage > 0) {
        const int lb = (stage - 1) & 1;
        ok = mbar_wait(lb ? mbar1 : mbar0, ph[lb]);
        if (!__syncthreads_and(ok ? 1 : 0)) bad = true;
    }
    fence_after_sync();
    __syncthreads();
    if (bad) {
        if (tid == 0) atomicExch(a.err, 1);
    } else {
        const int q = warp & 3, half = warp >> 2;
        const int row = q * 32 + lane, k = m0 + row;
        float* dst = a.partial + ((size_t)blockIdx.y * a.CO + (size_t)(k < a.CO ? k : 0)) * a.CI;
        for (int g = half; g < (a.NT >> 3); g += 2) {
            float v[8];
            if (stage > 0) {
                tmem_ld8(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g << 3), v);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = 0.f;
            }
            int c = n0 + (g << 3);
            if (k < a.CO && c < a.CI) {
                *reinterpret_cast<float4*>(dst + c) = make_float4(v[0], v[1], v[2], v[3]);
                *reinterpret_cast<float4*>(dst + c + 4) = make_float4(v[4], v[5], v[6], v[7]);
            }
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
    (void)pa; (void)pb;
}

__global__ void reduce_splits_tc(const float* __restrict__ partial, int splits, size_t n, float* __restrict__ out) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = 0.f;
    for (int k = 0; k < splits; ++k) s += partial[(size_t)k * n + i];
    out[i] = s;
}

struct Tiling {
    int NT, ntiles, KC, tmem_cols;
    size_t smem;
};

Tiling pick_tiling(int K, int N) {
    Tiling t;
    t.ntiles = (N + 255) / 256;
    t.NT = ((N + t.ntiles - 1) / t.ntiles + 15) / 16 * 16;
    t.ntiles = (N + t.NT - 1) / t.NT;
    int kpad = (K + KB - 1) / KB * KB;
    t.KC = kpad < 256 ? kpad : 256;
    t.tmem_cols = 32;
    while (t.tmem_cols < t.NT) t.tmem_cols <<= 1;
    t.smem = (size_t)(t.KC / KB) * (TM + t.NT) * 128 + 1024;
    return t;
}

template <bool BWD> void launch(const PwArgs& a0, const Tiling& t, int kind, double bytes, cudaStream_t st) {
    PwArgs a = a0;
    a.NT = t.NT; a.KC = t.KC; a.tmem_cols = t.tmem_cols;
    static bool attr_set = false;
    if (!attr_set) {
        cudaFuncSetAttribute(pw_tc_kernel<BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        attr_set = true;
    }
    LaunchScope ls(kind, bytes, 2.0 * a.P * a.N * a.K, st);
    dim3 grid((a.P + TM - 1) / TM, t.ntiles);
    pw_tc_kernel<BWD><<<grid, NTHREADS, t.smem, st>>>(a);
}

}  // namespace

bool pw_tc_supported(int dtype, const ConvGeom& g, bool bwd_data) {
    if (bwd_data && g.stride != 1) return false;
    return dtype == 1 && g.k == 1 && g.pad == 0 && g.ci % 8 == 0 && g.co % 8 == 0 && g.ci >= 8 && g.co >= 8;
}

void pw_fwd_tc(const ConvGeom& g, const ValSrc& x, const __nv_bfloat16* wb, const float* bias, void* z, int* err, cudaStream_t st) {
    PwArgs a{};
    a.x = x; a.w = wb; a.bias = bias; a.out = (__nv_bfloat16*)z; a.err = err;
    a.P = g.n * g.ho * g.wo; a.K = g.ci; a.N = g.co;
    a.stride = g.stride; a.ho = g.ho; a.wo = g.wo; a.hi = g.hi; a.wi = g.wi;
    Tiling t = pick_tiling(a.K, a.N);
    double bytes = 2.0 * ((double)a.P * a.K + (double)a.P * a.N) + 2.0 * a.N * a.K;
    launch<false>(a, t, K_PW_FWD_TC, bytes, st);
}

void pw_bwd_data_tc(const ConvGeom& g, const GradSrc& dz, const __nv_bfloat16* wtb, const void* addend, void* dx, int* err, cudaStream_t st) {
    PwArgs a{};
    a.dz = dz; a.w = wtb; a.addend = addend; a.out = (__nv_bfloat16*)dx; a.err = err;
    a.P = g.n * g.ho * g.wo; a.K = g.co; a.N = g.ci;
    a.stride = 1;
    Tiling t = pick_tiling(a.K, a.N);
    double bytes = 2.0 * (double)a.P * a.K * ((dz.act != ACT_NONE || dz.k1) ? 2.0 : 1.0) + 2.0 * (double)a.P * a.N * (addend ? 2.0 : 1.0) +
                   2.0 * a.N * a.K;
    launch<true>(a, t, K_PW_BWD_DATA_TC, bytes, st);
}

void pw_bwd_weight_tc(const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw, int* err,
                      cudaStream_t st) {
    PwWArgs a{};
    a.dz = dz; a.x = x; a.partial = scratch; a.err = err;
    a.P = g.n * g.ho * g.wo; a.CO = g.co; a.CI = g.ci;
    a.stride = g.stride; a.ho = g.ho; a.wo = g.wo; a.hi = g.hi; a.wi = g.wi;
    int ntiles = (a.CI + 255) / 256;
    a.NT = ((a.CI + ntiles - 1) / ntiles + 15) / 16 * 16;
    ntiles = (a.CI + a.NT - 1) / a.NT;
    a.tmem_cols = 32;
    while (a.tmem_cols < a.NT) a.tmem_cols <<= 1;
    int mtiles = (a.CO + TM - 1) / TM;
    size_t out_elems = (size_t)a.CO * a.CI;
    int splits = (2 * 148 + mtiles * ntiles - 1) / (mtiles * ntiles);
    int max_by_pix = (a.P + 4 * WSTAGE - 1) / (4 * WSTAGE);
    if (splits > max_by_pix) splits = max_by_pix;
    size_t cap = scratch_floats / out_elems;
    if ((size_t)splits > cap) splits = (int)cap;
    if (splits < 1) splits = 1;
    int ppc = (a.P + splits - 1) / splits;
    ppc = (ppc + WSTAGE - 1) / WSTAGE * WSTAGE;
    splits = (a.P + ppc - 1) / ppc;
    a.pix_per_cta = ppc;
    size_t smem = (size_t)2 * (2 + (a.NT + 63) / 64) * PANEL + 1024;
    static bool attr_set = false;
    if (!attr_set) {
        cudaFuncSetAttribute(pw_bwd_weight_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        attr_set = true;
    }
    double bytes = 2.0 * (double)a.P * a.CO * ((dz.act != ACT_NONE || dz.k1) ? 2.0 : 1.0) + 2.0 * (double)g.n * g.hi * g.wi * a.CI +
                   4.0 * out_elems * splits;
    {
        LaunchScope ls(K_PW_BWD_WEIGHT_TC, bytes, 2.0 * a.P * a.CO * a.CI, st);
        pw_bwd_weight_tc_kernel<<<dim3(mtiles, splits, ntiles), NTHREADS, smem, st>>>(a);
    }
    LaunchScope ls(K_REDUCE_SPLITS, 4.0 * out_elems * (splits + 1), (double)out_elems * splits, st);
    reduce_splits_tc<<<(unsigned)((out_elems + 255) / 256), 256, 0, st>>>(scratch, splits, out_elems, gw);
}

}  // namespace ast
