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
#include <string.h>

#include "kernels.h"
#include "tc_common.cuh"
#include "tma.cuh"

namespace ast {
namespace {

using namespace tc;
constexpr int NTHREADS = 256;

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

template <bool BWD> __global__ void __launch_bounds__(NTHREADS) pw_tc_kernel(const PwArgs a) {
    pdl_wait();
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t mbar_store;
    __shared__ uint32_t tmem_slot;
    __shared__ int failed;
    // 1024-byte aligned operand area (the swizzle pattern is a function of the address bits)
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
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
        // ---- stage A: [128 pixels][kc].  The global loads of four vectors per thread are issued together before any is
        // transformed, so that their latencies overlap instead of adding up. ----
        constexpr int U = 4;
        const bool need_z = BWD && grad_needs_z(a.dz);
        const int items = TM * vpr_pad;
        if (NTHREADS % vpr_pad == 0) {
            // usual case: the chunks per row divide the thread count, so a thread keeps one 16-byte channel chunk for the
            // whole reduction chunk and holds that chunk's transform coefficients in registers
            const int j = tid % vpr_pad, rstep = NTHREADS / vpr_pad;
            const bool data = j < vpr;
            const int c0 = k0 + ((data ? j : 0) << 3);
            XfVal xv;
            XfGrad xg;
            if (BWD) xg.init(a.dz, c0);
            else xv.init(a.x, c0);
            const uint4* src = reinterpret_cast<const uint4*>(BWD ? a.dz.dy : a.x.p);
            const uint4* srcz = reinterpret_cast<const uint4*>(a.dz.z);
            for (int rb = tid / vpr_pad; rb < TM; rb += U * rstep) {
                uint4 raw[U], rawz[U];
                bool ok[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = rb + u * rstep;
                    const int p = p0 + r;
                    ok[u] = r < TM && p < a.P && data;
                    raw[u] = rawz[u] = make_uint4(0, 0, 0, 0);
                    if (ok[u]) {
                        size_t pin = p;
                        if (!BWD && a.stride > 1) {
                            int wo = p % a.wo, t = p / a.wo;
                            int ho = t % a.ho, n = t / a.ho;
                            pin = ((size_t)n * a.hi + (size_t)ho * a.stride) * a.wi + (size_t)wo * a.stride;
                        }
                        const size_t e = (pin * a.K + c0) >> 3;
                        raw[u] = src[e];
                        if (need_z) rawz[u] = srcz[e];
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = rb + u * rstep;
                    if (r < TM) {
                        uint4 q = make_uint4(0, 0, 0, 0);
                        if (ok[u]) q = BWD ? (need_z ? xg.apply(raw[u], rawz[u]) : raw[u]) : xv.apply(raw[u]);
                        *reinterpret_cast<uint4*>(sA + tile_off(r, j, TM)) = q;
                    }
                }
            }
        } else
        for (int v0 = tid; v0 < items; v0 += U * NTHREADS) {
            Vec<__nv_bfloat16> raw[U], rawz[U];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * NTHREADS;
                const int r = v / vpr_pad, j = v - r * vpr_pad;
                const int p = p0 + r;
                ok[u] = v < items && p < a.P && j < vpr;
                raw[u].raw = rawz[u].raw = make_uint4(0, 0, 0, 0);
                if (ok[u]) {
                    const int c0 = k0 + (j << 3);
                    size_t pin = p;
                    if (!BWD && a.stride > 1) {
                        int wo = p % a.wo, t = p / a.wo;
                        int ho = t % a.ho, n = t / a.ho;
                        pin = ((size_t)n * a.hi + (size_t)ho * a.stride) * a.wi + (size_t)wo * a.stride;
                    }
                    const size_t e = (pin * a.K + c0) >> 3;
                    raw[u].load(BWD ? a.dz.dy : a.x.p, e);
                    if (need_z) rawz[u].load(a.dz.z, e);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * NTHREADS;
                if (v < items) {
                    const int r = v / vpr_pad, j = v - r * vpr_pad;
                    uint4 q = make_uint4(0, 0, 0, 0);
                    if (ok[u]) {
                        float f[8];
                        const int c0 = k0 + (j << 3);
                        if (BWD) grad_from_raw<__nv_bfloat16>(a.dz, raw[u], rawz[u], c0, f);
                        else val_from_raw<__nv_bfloat16>(a.x, raw[u], c0, f);
                        q = pack8(f);
                    }
                    *reinterpret_cast<uint4*>(sA + tile_off(r, j, TM)) = q;
                }
            }
        }
        // ---- stage B: [NT channels][kc] of the bf16 weights ----
#pragma unroll 4
        for (int v = tid; v < NT * vpr_pad; v += NTHREADS) {
            int r = v / vpr_pad, j = v - r * vpr_pad;
            int n = n0 + r;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (n < a.N && j < vpr) q = __ldg(reinterpret_cast<const uint4*>(a.w + (size_t)n * a.K + k0) + j);
            *reinterpret_cast<uint4*>(sB + tile_off(r, j, NT)) = q;
        }
        fence_async_smem();
        __syncthreads();
        if (warp == 0) {
            // the whole warp runs the issue loop in convergent control flow, the elected lane issues
            const uint32_t leader = elect_leader();
            fence_after_sync();
            const uint32_t a0 = smem_u32(sA), b0 = smem_u32(sB);
            const int steps = vpr_pad >> 1;           // 16 elements per MMA
            for (int s = 0; s < steps; ++s) {
                int kb = s >> 2, ks = s & 3;          // 64-element block, 32-byte step inside it
                uint64_t da = make_desc(a0 + (uint32_t)kb * TM * 128u + (uint32_t)ks * 32u);
                uint64_t db = make_desc(b0 + (uint32_t)kb * (uint32_t)NT * 128u + (uint32_t)ks * 32u);
                umma_bf16_lead(tmem, da, db, idesc, (k0 > 0 || s > 0) ? 1u : 0u, leader);
            }
            umma_commit_lead(mbar, leader);
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
        size_t pout = (size_t)p;
        if (BWD && a.stride > 1 && p < a.P) {      // gradient of a strided 1x1 conv lands on the sampled input pixels
            int wo = p % a.wo, t = p / a.wo;
            int ho = t % a.ho, n = t / a.ho;
            pout = ((size_t)n * a.hi + (size_t)ho * a.stride) * a.wi + (size_t)wo * a.stride;
        }
        // column groups in batches of four: the batch's residual-gradient loads are requested before its accumulators are read,
        // so that four loads are in flight instead of one dependent load per group
        for (int gb = half; gb < (NT >> 3); gb += 8) {
            Vec<__nv_bfloat16> av[4];
            if (BWD && a.addend) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int n = n0 + ((gb + 2 * u) << 3);
                    av[u].raw = make_uint4(0, 0, 0, 0);
                    if (gb + 2 * u < (NT >> 3) && p < a.P && n < a.N) av[u].load(a.addend, (pout * a.N + n) >> 3);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int g = gb + 2 * u;
                if (g >= (NT >> 3)) break;
                float v[8];
                tmem_ld8(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g << 3), v);
                int n = n0 + (g << 3);
                if (p < a.P && n < a.N) {
                    size_t e = pout * a.N + n;
                    if (!BWD && a.bias) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[i] += __ldg(a.bias + n + i);
                    }
                    if (BWD && a.addend) {
                        float ad[8];
                        av[u].unpack(ad);
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[i] += ad[i];
                    }
                    *reinterpret_cast<uint4*>(a.out + e) = pack8(v);
                }
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
    pdl_wait();
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t mbar_store[2];
    __shared__ uint32_t tmem_slot;
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
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
    const bool fast = ca > 0 && cb > 0 && NTHREADS % ca == 0 && NTHREADS % cb == 0;
    const int fja = fast ? tid % ca : 0, fjb = fast ? tid % cb : 0;
    XfGrad fxg;
    XfVal fxv;
    fxg.init(a.dz, m0 + (fja << 3));
    fxv.init(a.x, n0 + (fjb << 3));
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
        // both operands: the loads of four vectors per thread are issued together before any is transformed
        constexpr int U = 4;
        const bool need_z = grad_needs_z(a.dz);
        if (fast) {
            // a thread keeps one channel chunk of each operand; its coefficients were loaded into registers once
            const uint4* gdy = reinterpret_cast<const uint4*>(a.dz.dy);
            const uint4* gz = reinterpret_cast<const uint4*>(a.dz.z);
            const uint4* gx = reinterpret_cast<const uint4*>(a.x.p);
            for (int rb = tid / ca; rb < WSTAGE; rb += U * (NTHREADS / ca)) {
                uint4 raw[U], rawz[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int kr = rb + u * (NTHREADS / ca);
                    raw[u] = rawz[u] = make_uint4(0, 0, 0, 0);
                    if (kr < valid) {
                        const size_t e = ((size_t)(ps + kr) * a.CO + m0 + (fja << 3)) >> 3;
                        raw[u] = gdy[e];
                        if (need_z) rawz[u] = gz[e];
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int kr = rb + u * (NTHREADS / ca);
                    if (kr < WSTAGE) {
                        uint4 q = make_uint4(0, 0, 0, 0);
                        if (kr < valid) q = need_z ? fxg.apply(raw[u], rawz[u]) : raw[u];
                        *reinterpret_cast<uint4*>(sA + (fja >> 3) * PANEL + kr * 128 + (((fja & 7) ^ (kr & 7)) << 4)) = q;
                    }
                }
            }
            for (int rb = tid / cb; rb < WSTAGE; rb += U * (NTHREADS / cb)) {
                uint4 raw[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int kr = rb + u * (NTHREADS / cb);
                    raw[u] = make_uint4(0, 0, 0, 0);
                    if (kr < valid) {
                        size_t pin = ps + kr;
                        if (a.stride > 1) {
                            int p = ps + kr;
                            int wo = p % a.wo, t = p / a.wo;
                            int ho = t % a.ho, n = t / a.ho;
                            pin = ((size_t)n * a.hi + (size_t)ho * a.stride) * a.wi + (size_t)wo * a.stride;
                        }
                        raw[u] = gx[(pin * a.CI + n0 + (fjb << 3)) >> 3];
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int kr = rb + u * (NTHREADS / cb);
                    if (kr < WSTAGE) {
                        const uint4 q = kr < valid ? fxv.apply(raw[u]) : make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4*>(sB + (fjb >> 3) * PANEL + kr * 128 + (((fjb & 7) ^ (kr & 7)) << 4)) = q;
                    }
                }
            }
        } else {
        for (int v0 = tid; v0 < WSTAGE * ca; v0 += U * NTHREADS) {
            Vec<__nv_bfloat16> raw[U], rawz[U];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * NTHREADS;
                const int kr = v / ca, j = v - kr * ca;
                ok[u] = v < WSTAGE * ca && kr < valid;
                raw[u].raw = rawz[u].raw = make_uint4(0, 0, 0, 0);
                if (ok[u]) {
                    const size_t e = ((size_t)(ps + kr) * a.CO + m0 + (j << 3)) >> 3;
                    raw[u].load(a.dz.dy, e);
                    if (need_z) rawz[u].load(a.dz.z, e);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * NTHREADS;
                if (v < WSTAGE * ca) {
                    const int kr = v / ca, j = v - kr * ca;
                    uint4 q = make_uint4(0, 0, 0, 0);
                    if (ok[u]) {
                        float f[8];
                        grad_from_raw<__nv_bfloat16>(a.dz, raw[u], rawz[u], m0 + (j << 3), f);
                        q = pack8(f);
                    }
                    *reinterpret_cast<uint4*>(sA + (j >> 3) * PANEL + kr * 128 + (((j & 7) ^ (kr & 7)) << 4)) = q;
                }
            }
        }
        for (int v0 = tid; v0 < WSTAGE * cb; v0 += U * NTHREADS) {
            Vec<__nv_bfloat16> raw[U];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * NTHREADS;
                const int kr = v / cb, j = v - kr * cb;
                ok[u] = v < WSTAGE * cb && kr < valid;
                raw[u].raw = make_uint4(0, 0, 0, 0);
                if (ok[u]) {
                    size_t pin = ps + kr;
                    if (a.stride > 1) {
                        int p = ps + kr;
                        int wo = p % a.wo, t = p / a.wo;
                        int ho = t % a.ho, n = t / a.ho;
                        pin = ((size_t)n * a.hi + (size_t)ho * a.stride) * a.wi + (size_t)wo * a.stride;
                    }
                    raw[u].load(a.x.p, (pin * a.CI + n0 + (j << 3)) >> 3);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * NTHREADS;
                if (v < WSTAGE * cb) {
                    const int kr = v / cb, j = v - kr * cb;
                    uint4 q = make_uint4(0, 0, 0, 0);
                    if (ok[u]) {
                        float f[8];
                        val_from_raw<__nv_bfloat16>(a.x, raw[u], n0 + (j << 3), f);
                        q = pack8(f);
                    }
                    *reinterpret_cast<uint4*>(sB + (j >> 3) * PANEL + kr * 128 + (((j & 7) ^ (kr & 7)) << 4)) = q;
                }
            }
        }
        }
        fence_async_smem();
        __syncthreads();
        if (warp == 0) {
            const uint32_t leader = elect_leader();
            fence_after_sync();
            const uint32_t a0 = smem_u32(sA), b0 = smem_u32(sB);
#pragma unroll
            for (int s = 0; s < WSTAGE / 16; ++s)      // 16 pixels = two 8-row groups per MMA
                umma_bf16_lead(tmem, make_desc_mn(a0 + s * 2048), make_desc_mn(b0 + s * 2048), idesc, (stage > 0 || s > 0) ? 1u : 0u, leader);
            umma_commit_lead(b ? mbar1 : mbar0, leader);
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


// ---------------------------------------------------------------------------------------------
// Persistent, warp-specialised form of the forward / backward-data GEMM (one CTA per SM).
//
//   warp 0      producer: bulk-copies (cp.async.bulk, completion on an mbarrier) the raw tile
//               rows [pixels][K] of x (forward) or of dy and z (backward) into a ring of
//               shared-memory stages; a tile of consecutive pixels is one contiguous byte range
//   warp 1      MMA issuer: tcgen05.mma over the staged operand into one of two accumulators in
//               tensor memory; tcgen05.commit releases the operand stage and publishes the tile
//   warps 2-9   transformers: read a raw stage, apply BatchNorm+activation (or the
//               BatchNorm-backward transform) with per-thread register-held coefficients,
//               write bf16 into the swizzled K-major operand stage
//   warps 10-13 epilogue: tcgen05.ld the finished accumulator, add bias / residual gradient,
//               store bf16 to global
//
// Copy, transform, MMA and store of consecutive tiles overlap.  The weights stay resident in
// shared memory.  Every wait is bounded; a wait that runs out raises a CTA-wide abort flag, every
// role leaves its loop, outstanding bulk copies are waited for, tensor memory is freed and the
// error word is set.
constexpr int PIPE_WORKERS = 12;      // transform + epilogue warps
constexpr int PIPE_THREADS = (2 + PIPE_WORKERS) * 32;     // producer, MMA issuer, workers
constexpr int MAX_RAW = 8;

struct PipeArgs {
    ValSrc x;
    GradSrc dz;
    const __nv_bfloat16* w;     // [N][K]
    const float* bias;
    const void* addend;
    __nv_bfloat16* out;
    int* err;
    int P, K, N, NT, tiles;
    int tmem_cols;
    int RS, R;                  // raw stage: RS pixels (divides 128); ring of R stages
    int need_z;                 // backward: the transform also reads z
    uint32_t raw_bytes;         // bytes of one raw stage (both tensors), multiple of 128
    uint32_t a_bytes, b_bytes;  // one operand stage / the resident weights
    uint32_t o_bytes;           // one output staging tile
    int panels;                 // staging tile layout: 1 = 64-channel panels of [128 rows][128 bytes], 16-byte chunks XOR-swizzled with the
                                // row, stored by tiled tensor copies (N a multiple of 64); 0 = [128][N] row-major, stored by one bulk copy
    uint32_t z_bytes;           // one tile [128][N] bf16 of the producing unit's raw output (backward sums), multiple of 128
    int OS;                     // output staging tiles: 1 or 2
    int AS;                     // operand stages: 2, or 1 where a long reduction leaves no room for two
    int xf_warps;               // of the 12 worker warps, how many transform (4 or 8); the rest run the epilogue: a tile
                                // costs the transform warps ~K and the epilogue warps ~N instructions per row
    const float* pivot;         // forward, optional: per-channel pivot of the fused BatchNorm statistics
    float* stat_partial;        // [CTAs][2][N]: sums of (z - pivot) and (z - pivot)^2 over the CTA's pixels
    // backward, optional: BatchNorm-backward sums of the produced gradient (the unit that made this conv's input)
    const __nv_bfloat16* rz;    // that unit's raw output [P][N]
    const float *r_scale, *r_shift, *r_mean, *r_rstd;
    int r_act;
    float* r_partial;           // [CTAs][2][N]: sums of dpre and dpre * xhat over the CTA's pixels
};

// EXTRA: the epilogue adds the bias (forward) or the residual gradient (backward); a template
// parameter because even a never-taken branch around those loads slows the epilogue's inner loop.
// PANELS: layout of the output staging tile (see PipeArgs::panels); a template parameter for the same reason.
template <bool BWD, bool EXTRA, bool PANELS> __global__ void __launch_bounds__(PIPE_THREADS, 1) pw_pipe_kernel(const __grid_constant__ CUtensorMap tm_out, const PipeArgs a) {
    // Set-up that reads nothing the previous kernel in the stream writes (barriers, tensor memory, the resident
    // weights: written only by the refresh kernel, which never releases its dependents before it has completed) runs before
    // the dependency wait and so overlaps the previous kernel's tail.
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    // raw_full[R], raw_empty[R], a_full[2], a_empty[2], acc_full[2], acc_empty[2], zp_full[2], zp_empty[2], so_full[2], so_free[2]
    __shared__ uint64_t bars[2 * MAX_RAW + 16];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_store;
    volatile int* abort_flag = &abort_store;
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* sA = base;                               // operand stages (a.AS of them)
    uint8_t* sB = base + (size_t)a.AS * a.a_bytes;    // resident weights
    uint8_t* sO = sB + a.b_bytes;                     // output staging tiles (1024-byte aligned: the swizzle is a function of the address)
    uint8_t* sR = sO + (size_t)a.OS * a.o_bytes;      // raw ring
    uint8_t* sZ = sR + (size_t)a.R * a.raw_bytes;     // backward sums: two tiles of the producing unit's raw output
    const bool bred = BWD && a.r_partial != nullptr;
    const bool csum = bred || (!BWD && a.stat_partial != nullptr);   // the transform warps take column sums of every output tile
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = a.R, RS = a.RS, subs = TM / RS;
    const int nxf = a.xf_warps * 32, nepi = (PIPE_WORKERS - a.xf_warps) * 32, epi_warp0 = 2 + a.xf_warps;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto raw_full = [&](int s) { return bar0 + 8u * s; };
    auto raw_empty = [&](int s) { return bar0 + 8u * (MAX_RAW + s); };
    auto a_full = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + s); };
    auto a_empty = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + 2 + s); };
    auto acc_full = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + 4 + s); };
    auto acc_empty = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + 6 + s); };
    auto zp_full = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + 8 + s); };
    auto zp_empty = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + 10 + s); };
    auto so_full = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + 12 + s); };
    auto so_free = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + 14 + s); };

    if (tid == 0) {
        for (int s = 0; s < R; ++s) {
            mbar_init(raw_full(s), 1);
            mbar_init(raw_empty(s), a.xf_warps);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(a_full(s), a.xf_warps);
            mbar_init(a_empty(s), 1);
            mbar_init(acc_full(s), 1);
            mbar_init(acc_empty(s), PIPE_WORKERS - a.xf_warps);
            mbar_init(zp_full(s), 1);
            mbar_init(zp_empty(s), a.xf_warps);
            mbar_init(so_full(s), 1);
            mbar_init(so_free(s), a.xf_warps);
        }
        abort_store = 0;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), (uint32_t)a.tmem_cols);
        tmem_relinquish();
    }
    const int NT = a.NT;
    const int vpr = a.K >> 3, vpr_pad = ((a.K + 15) >> 4) << 1;
    // resident weights: [NT][K] bf16 -> swizzled K-major blocks (rows beyond N and the K padding are zero)
    for (int v = tid; v < NT * vpr_pad; v += PIPE_THREADS) {
        int r = v / vpr_pad, j = v - r * vpr_pad;
        uint4 q = make_uint4(0, 0, 0, 0);
        if (r < a.N && j < vpr) q = __ldg(reinterpret_cast<const uint4*>(a.w + (size_t)r * a.K) + j);
        *reinterpret_cast<uint4*>(sB + tile_off(r, j, NT)) = q;
    }
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    pdl_wait();
    const uint32_t tmem = tmem_slot;
    const int my_tiles = (a.tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const uint32_t row_bytes = (uint32_t)a.K * 2u;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            const uint8_t* src0 = reinterpret_cast<const uint8_t*>(BWD ? a.dz.dy : a.x.p);
            const uint8_t* src1 = reinterpret_cast<const uint8_t*>(a.dz.z);
            int it = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tile = blockIdx.x + t * gridDim.x;
                for (int sub = 0; sub < subs; ++sub, ++it) {
                    const int s = it % R, n = it / R;
                    if (n > 0 && !mbar_wait_abortable(raw_empty(s), (uint32_t)((n - 1) & 1), abort_flag)) {
                        ok = false;
                        break;
                    }
                    const int p_first = tile * TM + sub * RS;
                    int valid = a.P - p_first;
                    valid = valid < 0 ? 0 : (valid > RS ? RS : valid);
                    const uint32_t bytes = (uint32_t)valid * row_bytes;
                    uint8_t* dst = sR + (size_t)s * a.raw_bytes;
                    if (valid > 0) {
                        mbar_expect_tx(raw_full(s), bytes * ((BWD && a.need_z) ? 2u : 1u));
                        bulk_g2s(smem_u32(dst), src0 + (size_t)p_first * row_bytes, bytes, raw_full(s));
                        if (BWD && a.need_z) bulk_g2s(smem_u32(dst + (size_t)RS * row_bytes), src1 + (size_t)p_first * row_bytes, bytes, raw_full(s));
                    } else {
                        mbar_arrive(raw_full(s));
                    }
                }
            }
            // never leave while a bulk copy into this CTA's shared memory may still be in flight
            const int issued = it;
            for (int k = (issued > R ? issued - R : 0); k < issued; ++k) mbar_wait(raw_full(k % R), (uint32_t)((k / R) & 1));
        } else if (lane == 1 && bred) {
            // second copy stream (its own thread, so that waiting for a free tile buffer never holds back the raw
            // ring's prefetch): for every output tile, the matching tile of the producing unit's raw output
            int zissued = 0;
            for (int t = 0; t < my_tiles; ++t, ++zissued) {
                const int tile = blockIdx.x + t * gridDim.x;
                const int zb = t & 1, zn = t >> 1;
                if (zn > 0 && !mbar_wait_abortable(zp_empty(zb), (uint32_t)((zn - 1) & 1), abort_flag)) break;
                const int valid = min(TM, a.P - tile * TM);
                const uint32_t bytes = (uint32_t)valid * (uint32_t)a.N * 2u;
                mbar_expect_tx(zp_full(zb), bytes);
                bulk_g2s(smem_u32(sZ + (size_t)zb * a.z_bytes), a.rz + (size_t)tile * TM * a.N, bytes, zp_full(zb));
            }
            for (int k = (zissued > 2 ? zissued - 2 : 0); k < zissued; ++k) mbar_wait(zp_full(k & 1), (uint32_t)((k >> 1) & 1));
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        // every lane runs the loop (convergent control flow keeps the descriptor arithmetic in the uniform datapath: a
        // single diverged lane issues at about half the rate), the elected lane issues
        {
            const uint32_t leader = elect_leader();
            const uint32_t idesc = make_idesc(NT);
            const uint64_t dconst = make_desc(0);
            const uint32_t a0 = smem_u32(sA) >> 4, b0 = smem_u32(sB) >> 4;
            const int steps = vpr_pad >> 1;
            for (int t = 0; t < my_tiles; ++t) {
                const int st = t & 1, n = t >> 1;                                    // accumulator stage and its use count
                const int as = a.AS == 2 ? (t & 1) : 0, an = a.AS == 2 ? (t >> 1) : t;   // operand stage and its use count
                if (!mbar_wait_abortable(a_full(as), (uint32_t)(an & 1), abort_flag)) break;
                if (n > 0 && !mbar_wait_abortable(acc_empty(st), (uint32_t)((n - 1) & 1), abort_flag)) break;
                fence_after_sync();
                const uint32_t d = tmem + (uint32_t)(st * NT);
                const uint32_t as0 = a0 + ((uint32_t)as * a.a_bytes >> 4);
                for (int k = 0; k < steps; ++k) {
                    const uint32_t kb = (uint32_t)k >> 2, ks = (uint32_t)k & 3u;
                    umma_bf16_lead(d, dconst + (uint64_t)(as0 + kb * (TM * 8u) + ks * 2u), dconst + (uint64_t)(b0 + kb * ((uint32_t)NT * 8u) + ks * 2u), idesc,
                                   k > 0 ? 1u : 0u, leader);
                }
                umma_commit_lead(a_empty(as), leader);
                umma_commit_lead(acc_full(st), leader);
                __syncwarp();
            }
        }
    } else if (warp < epi_warp0) {
        // ------------------------------------------------------------ transformers
        const int tix = tid - 64;
        const int groups = nxf / vpr_pad;                 // row groups; thread (grp, j) owns chunk j of rows grp, grp+groups, ...
        const int j = tix % vpr_pad, grp = tix / vpr_pad;
        const bool active = grp < groups;
        const bool data = j < vpr;                        // chunks beyond K are zero padding
        const int c0 = data ? (j << 3) : 0;
        XfVal xv;
        XfGrad xg;
        if (BWD) xg.init(a.dz, c0);
        else xv.init(a.x, c0);
        // Column sums (optional): the transform warps also take, for every finished output tile, per-channel sums down the
        // staged (rounded) tile; thread (cu, rh) owns four channels and the rows rh, rh + r_split, ...
        //   forward:  sums of (z - pivot) and (z - pivot)^2, the BatchNorm statistics partials of the output;
        //   backward: sums of dpre = dx * [pre inside the activation's linear region] and dpre * xhat, with pre = z*rcs + rch
        //             and xhat = z*rrs + rms taken from the matching tile of the producing unit's raw output z.
        const int r_units = a.N >> 2, r_split = nxf / r_units;
        const int cu = tix % r_units, rh = tix / r_units;
        const bool ractive = csum && rh < r_split;
        float s1[4], s2[4], rcs[4], rch[4], rrs[4], rms[4];     // forward: rcs holds the pivot
        const float rlo = a.r_act == ACT_NONE ? -INFINITY : 0.f, rhi = a.r_act == ACT_RELU6 ? 6.f : INFINITY;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            s1[i] = s2[i] = 0.f;
            if (BWD) {
                rcs[i] = ractive ? __ldg(a.r_scale + cu * 4 + i) : 1.f;
                rch[i] = ractive ? __ldg(a.r_shift + cu * 4 + i) : 0.f;
                rrs[i] = ractive ? __ldg(a.r_rstd + cu * 4 + i) : 0.f;
                rms[i] = ractive ? -__ldg(a.r_mean + cu * 4 + i) * rrs[i] : 0.f;
            } else {
                rcs[i] = ractive ? __ldg(a.pivot + cu * 4 + i) : 0.f;
            }
        }
        auto reduce_tile = [&](int r) -> bool {
            const int ob = a.OS == 2 ? (r & 1) : 0, zb = r & 1;
            bool got = mbar_wait_abortable(so_full(ob), (uint32_t)((r / a.OS) & 1), abort_flag);
            if (BWD) got = got && mbar_wait_abortable(zp_full(zb), (uint32_t)((r >> 1) & 1), abort_flag);
            if (got && ractive) {
                const uint32_t row_out = (uint32_t)a.N * 2u;
                const uint8_t* so = sO + (size_t)ob * a.o_bytes;
                const uint8_t* sz = sZ + (size_t)zb * a.z_bytes;
                // the thread's four channels inside the staged tile: panel, 16-byte chunk, half of the chunk
                const uint32_t so_col = (uint32_t)(cu >> 4) * (TM * 128u) + (uint32_t)((cu & 1) << 3);
                const uint32_t so_chunk = (uint32_t)((cu & 15) >> 1);
                const int valid = min(TM, a.P - ((int)blockIdx.x + r * (int)gridDim.x) * TM);
#pragma unroll 2
                for (int rr = rh; rr < valid; rr += r_split) {
                    const uint2 dr = PANELS ? *reinterpret_cast<const uint2*>(so + so_col + (uint32_t)rr * 128u + ((so_chunk ^ (uint32_t)(rr & 7)) << 4))
                                              : *reinterpret_cast<const uint2*>(so + (size_t)rr * row_out + (cu << 3));
                    const float d[4] = {__uint_as_float(dr.x << 16), __uint_as_float(dr.x & 0xffff0000u), __uint_as_float(dr.y << 16),
                                        __uint_as_float(dr.y & 0xffff0000u)};
                    if (BWD) {
                        const uint2 zr = *reinterpret_cast<const uint2*>(sz + (size_t)rr * row_out + (cu << 3));
                        const float z[4] = {__uint_as_float(zr.x << 16), __uint_as_float(zr.x & 0xffff0000u), __uint_as_float(zr.y << 16),
                                            __uint_as_float(zr.y & 0xffff0000u)};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float pre = fmaf(z[i], rcs[i], rch[i]);
                            const float dm = (pre > rlo && pre < rhi) ? d[i] : 0.f;
                            s1[i] += dm;
                            s2[i] = fmaf(dm, fmaf(z[i], rrs[i], rms[i]), s2[i]);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float dd = d[i] - rcs[i];
                            s1[i] += dd;
                            s2[i] = fmaf(dd, dd, s2[i]);
                        }
                    }
                }
            }
            // one arrival per warp (an arrival is a shared-memory atomic: hundreds of them per hand-off serialise)
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(so_free(ob));
                if (BWD) mbar_arrive(zp_empty(zb));
            }
            return got;
        };
        int it = 0, reduced_tiles = 0;
        bool ok = true;
        for (int t = 0; t < my_tiles && ok; ++t) {
            const int tile = blockIdx.x + t * gridDim.x;
            const int st = a.AS == 2 ? (t & 1) : 0, n = a.AS == 2 ? (t >> 1) : t;    // operand stage and its use count
            if (n > 0 && !mbar_wait_abortable(a_empty(st), (uint32_t)((n - 1) & 1), abort_flag)) break;
            uint8_t* dstA = sA + (size_t)st * a.a_bytes;
            for (int sub = 0; sub < subs; ++sub, ++it) {
                const int s = it % R;
                if (!mbar_wait_abortable(raw_full(s), (uint32_t)((it / R) & 1), abort_flag)) {
                    ok = false;
                    break;
                }
                const uint8_t* raw = sR + (size_t)s * a.raw_bytes;
                if (active) {
                    // straight-line body (rows past the end of the tensor and the K padding are
                    // read like any other and zeroed afterwards) so that the unrolled iterations'
                    // loads and arithmetic interleave
                    const int jl = data ? j : 0;
                    const int rows_left = a.P - tile * TM - sub * RS;
                    // not unrolled: the kernel's roles share a small instruction cache, and this loop gains nothing from a
                    // longer body (a load cannot move above a store that might alias it)
#pragma unroll 1
                    for (int rl = grp; rl < RS; rl += groups) {
                        const uint4 r0 = *reinterpret_cast<const uint4*>(raw + (size_t)rl * row_bytes + (jl << 4));
                        uint4 q4;
                        if (!BWD) {
                            q4 = xv.apply(r0);
                        } else if (a.need_z) {
                            q4 = xg.apply(r0, *reinterpret_cast<const uint4*>(raw + (size_t)(RS + rl) * row_bytes + (jl << 4)));
                        } else {
                            q4 = r0;
                        }
                        if (!data || rl >= rows_left) q4 = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4*>(dstA + tile_off(sub * RS + rl, j, TM)) = q4;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(raw_empty(s));
            }
            if (!ok) break;
            fence_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(a_full(st));
            // as many tiles behind as there are staging tiles: by then that tile's MMA and epilogue have had the time of
            // a whole transform + sum step, and the staging tile it occupies is the next one the epilogue needs back
            if (csum && t >= a.OS) {
                ok = reduce_tile(reduced_tiles);
                ++reduced_tiles;
            }
        }
        if (csum) {
            while (ok && reduced_tiles < my_tiles) {
                ok = reduce_tile(reduced_tiles);
                ++reduced_tiles;
            }
            // combine the r_split row classes of every column group in fixed order (every transform thread gets here,
            // also after an abort: all waits are bounded); the operand stages are free now: the last tile's sums were
            // taken after its epilogue, hence after its MMAs
            named_bar_sync(2, nxf);
            float* red = reinterpret_cast<float*>(sA);        // [r_split][2][N]
            if (ractive) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    red[(rh * 2 + 0) * a.N + cu * 4 + i] = s1[i];
                    red[(rh * 2 + 1) * a.N + cu * 4 + i] = s2[i];
                }
            }
            named_bar_sync(2, nxf);
            for (int e = tix; e < 2 * a.N; e += nxf) {
                float acc = 0.f;
                for (int k = 0; k < r_split; ++k) acc += red[k * 2 * a.N + e];
                (BWD ? a.r_partial : a.stat_partial)[(size_t)blockIdx.x * 2 * a.N + e] = acc;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        // The epilogue threads (one accumulator row each) round the tile to bf16 into a shared-memory
        // staging tile.  With N a multiple of 64 the tile is made of 64-channel panels whose rows are
        // 128 bytes with the 16-byte chunks XOR-swizzled by the row index: the 32 rows a warp stores at
        // once then fall into different banks (a row-major tile puts them all into the same four), and
        // one thread hands the panels to tiled tensor copies that undo the swizzle on the way to global
        // memory.  Other widths keep the row-major tile, which is the output's own byte range and
        // leaves with a single bulk copy.
        const int q = warp & 3;                            // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;
        const int et = tid - epi_warp0 * 32;
        const int half = (warp - epi_warp0) >> 2, nhalf = nepi >> 7;      // several threads share a row: they alternate column batches
        const uint32_t row_out = (uint32_t)a.N * 2u;
        int issued = 0;
        for (int t = 0; t < my_tiles; ++t) {
            const int tile = blockIdx.x + t * gridDim.x;
            const int st = t & 1, n = t >> 1;
            const int ob = a.OS == 2 ? (t & 1) : 0;
            uint8_t* so = sO + (size_t)ob * a.o_bytes;
            bool ok = mbar_wait_abortable(acc_full(st), (uint32_t)(n & 1), abort_flag);
            // the transform warps must have finished the column sums over this staging tile's previous contents
            if (csum && t >= a.OS) ok = mbar_wait_abortable(so_free(ob), (uint32_t)((t / a.OS - 1) & 1), abort_flag) && ok;
            // the bulk store that last read this staging tile must have finished reading it
            if (et == 0) {
                if (a.OS == 2) bulk_wait_read<1>();
                else bulk_wait_read<0>();
            }
            ok = named_bar_and(1, nepi, ok);
            if (!ok) break;
            fence_after_sync();
            const int p = tile * TM + row;
            // accumulator columns in batches of up to 64: the batch's tcgen05.ld are all issued
            // before the one wait, so their latencies overlap
            for (int g0 = half * 4; g0 < (NT >> 4); g0 += 4 * nhalf) {
                uint32_t rr[4][16];
                // the residual gradient of the batch's 64 columns is requested before the accumulators are read: eight loads in
                // flight beside the tcgen05.ld instead of one dependent load per 8 columns
                Vec<__nv_bfloat16> adv[4][2];
                if (BWD && EXTRA) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            const int nn = ((g0 + u) << 4) + (hh << 3);
                            adv[u][hh].raw = make_uint4(0, 0, 0, 0);
                            if (p < a.P && nn < a.N) adv[u][hh].load(a.addend, ((size_t)p * a.N + nn) >> 3);
                        }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (g0 + u < (NT >> 4)) tmem_ld16_issue(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(st * NT + ((g0 + u) << 4)), rr[u]);
                tmem_ld_wait();
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (g0 + u < (NT >> 4)) tmem_ld_pin16(rr[u]);
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const int nn = ((g0 + u) << 4) + (hh << 3);
                        if (nn < a.N) {
                            float vv[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) vv[i] = __uint_as_float(rr[u][(hh << 3) + i]);
                            if (!BWD && EXTRA) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) vv[i] += __ldg(a.bias + nn + i);
                            }
                            if (BWD && EXTRA && p < a.P) {
                                float ad[8];
                                adv[u][hh].unpack(ad);
#pragma unroll
                                for (int i = 0; i < 8; ++i) vv[i] += ad[i];
                            }
                            const uint32_t so_off = PANELS ? (uint32_t)(nn >> 6) * (TM * 128u) + (uint32_t)row * 128u + ((((uint32_t)(nn & 63) >> 3) ^ (uint32_t)(row & 7)) << 4)
                                                             : (uint32_t)row * row_out + (uint32_t)(nn << 1);
                            *reinterpret_cast<uint4*>(so + so_off) = pack8(vv);
                        }
                    }
                }
            }
            fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(st));
            fence_async_smem();
            named_bar_sync(1, nepi);
            if (et == 0) {
                if (PANELS) {
                    // rows past the end of the tensor are clipped by the copy
                    for (int pn = 0; pn * 64 < a.N; ++pn) tma::store_2d(&tm_out, smem_u32(so) + (uint32_t)pn * (TM * 128u), pn * 64, tile * TM);
                } else {
                    bulk_s2g(a.out + (size_t)tile * TM * a.N, smem_u32(so), (uint32_t)min(TM, a.P - tile * TM) * row_out);
                }
                bulk_commit();
                ++issued;
                if (csum) mbar_arrive(so_full(ob));      // the staged tile is complete (ordered by the named barrier above)
            }
        }
        if (et == 0 && issued > 0) bulk_wait<0>();
    }
    fence_before_sync();
    __syncthreads();
    if (tid == 0 && abort_store) atomicExch(a.err, 1);
    if (warp == 1) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
}

// Chooses the pipeline's shared-memory split; returns false if the shape does not fit (large K
// or N), in which case the one-tile-per-CTA kernel is used.
bool plan_pipe(PipeArgs& a, size_t* smem) {
    if (a.N > 256 || a.K > 256) return false;
    a.NT = (a.N + 15) / 16 * 16;
    a.tmem_cols = 32;
    while (a.tmem_cols < 2 * a.NT) a.tmem_cols <<= 1;
    if (a.tmem_cols > 512) return false;
    const int nkb = (a.K + KB - 1) / KB;
    a.a_bytes = (uint32_t)nkb * TM * 128u;
    a.b_bytes = (uint32_t)nkb * (uint32_t)a.NT * 128u;
    a.z_bytes = ((uint32_t)TM * (uint32_t)a.N * 2u + 127u) / 128u * 128u;
    a.panels = a.N % 64 == 0 ? 1 : 0;
    a.o_bytes = a.panels ? (uint32_t)(a.N / 64) * TM * 128u : (a.z_bytes + 1023u) / 1024u * 1024u;
    const size_t budget = 220 * 1024 - 1024;
    const int tensors = a.need_z ? 2 : 1;
    const size_t zp = a.r_partial ? 2 * (size_t)a.z_bytes : 0;      // two tiles of the raw output the backward sums read
    // two operand stages if they fit; one for long reductions (the transform of tile t+1 then waits for the MMAs of t)
    {
        // split of the twelve worker warps: estimated instructions per tile of the two roles, spread over their warps
        const double vpr_pad = ((a.K + 15) / 16) * 2;
        const bool csum = a.stat_partial != nullptr || a.r_partial != nullptr;
        const double xf_work = 128.0 * vpr_pad * (a.need_z ? 60.0 : 30.0) + (csum ? 128.0 * (a.N / 4) * (a.r_partial ? 25.0 : 15.0) : 0.0);
        const double epi_work = 128.0 * (a.N / 8.0) * ((a.addend || a.bias) ? 35.0 : 22.0);
        double best = 0;
        a.xf_warps = 8;
        for (int x = 4; x <= PIPE_WORKERS - 4; x += 4) {
            const double t = xf_work / x > epi_work / (PIPE_WORKERS - x) ? xf_work / x : epi_work / (PIPE_WORKERS - x);
            if (x == 4 || t < best) {
                best = t;
                a.xf_warps = x;
            }
        }
    }
    for (a.AS = 2; a.AS >= 1; --a.AS) {
        const size_t ab = (size_t)a.AS * a.a_bytes;
        // two output staging tiles if that still leaves room for two 64-pixel raw stages
        a.OS = ab + a.b_bytes + 2 * (size_t)a.o_bytes + zp + 2 * (((size_t)64 * a.K * 2 * tensors + 127) / 128 * 128) <= budget ? 2 : 1;
        const size_t fixed = ab + a.b_bytes + (size_t)a.OS * a.o_bytes + zp;
        if (fixed >= budget) continue;
        for (int rs = 128; rs >= 32; rs >>= 1) {
            size_t rb = ((size_t)rs * a.K * 2 * tensors + 127) / 128 * 128;
            size_t r = (budget - fixed) / rb;
            if (r >= 2) {
                // at least two stages in flight, at most MAX_RAW and no more than three tiles' worth
                size_t cap = (size_t)3 * (TM / rs);
                if (r > cap) r = cap;
                if (r > MAX_RAW) r = MAX_RAW;
                a.RS = rs;
                a.R = (int)r;
                a.raw_bytes = (uint32_t)rb;
                *smem = fixed + r * rb + 1024;
                return true;
            }
        }
    }
    return false;
}

// tensor map of the output [P][N] for the epilogue's panel stores: boxes of 64 channels x 128 pixels
bool make_out_map(const void* out, int P, int N, CUtensorMap* m) {
    const uint64_t dims[2] = {(uint64_t)N, (uint64_t)P};
    const uint64_t strides[1] = {(uint64_t)N * 2};
    const uint32_t box[2] = {64, TM};
    return tma::encode_bf16(m, out, 2, dims, strides, box);
}

template <bool BWD> int launch_pipe(PipeArgs& a, const CUtensorMap& tm_out, size_t smem, int kind, double bytes, size_t partial_floats, cudaStream_t st) {
    smem_limit_once<101 + (BWD ? 50 : 0)>(pw_pipe_kernel<BWD, false, false>, 222 * 1024);
    smem_limit_once<102 + (BWD ? 50 : 0)>(pw_pipe_kernel<BWD, true, false>, 222 * 1024);
    smem_limit_once<103 + (BWD ? 50 : 0)>(pw_pipe_kernel<BWD, false, true>, 222 * 1024);
    smem_limit_once<104 + (BWD ? 50 : 0)>(pw_pipe_kernel<BWD, true, true>, 222 * 1024);
    const int n_sm = sm_count();
    int grid = a.tiles < n_sm ? a.tiles : n_sm;
    if (a.stat_partial && (size_t)grid * 2 * a.N > partial_floats) a.stat_partial = nullptr;
    if (a.r_partial && (size_t)grid * 2 * a.N > partial_floats) a.r_partial = nullptr;
    const bool fused = BWD ? a.r_partial != nullptr : a.stat_partial != nullptr;
    LaunchScope ls(kind, bytes + (fused ? 8.0 * a.N * grid : 0.0) + (BWD && fused ? 2.0 * a.P * a.N : 0.0), 2.0 * a.P * a.N * a.K, st);
    const bool extra = BWD ? a.addend != nullptr : a.bias != nullptr;
    if (a.panels) {
        if (extra) launch_pdl(pw_pipe_kernel<BWD, true, true>, grid, PIPE_THREADS, smem, st, tm_out, a);
        else launch_pdl(pw_pipe_kernel<BWD, false, true>, grid, PIPE_THREADS, smem, st, tm_out, a);
    } else {
        if (extra) launch_pdl(pw_pipe_kernel<BWD, true, false>, grid, PIPE_THREADS, smem, st, tm_out, a);
        else launch_pdl(pw_pipe_kernel<BWD, false, false>, grid, PIPE_THREADS, smem, st, tm_out, a);
    }
    return fused ? grid : 0;
}


// ---------------------------------------------------------------------------------------------
// Pipelined weight gradient (one CTA per pixel range, all output channels in one CTA).
//
//   warp 0      producer: per 64-pixel stage, bulk-copies the raw rows of dy, z and x
//   warp 1      MMA issuer: for every (128-row, N-tile) pair one tcgen05.mma per 16 pixels into
//               its own tensor-memory columns, accumulating over the CTA's whole pixel range
//   warps 2-9   transformers: dz = BatchNorm/activation backward of (dy, z), x = BatchNorm +
//               activation of the producer's raw output, both written bf16 MN-major; after the
//               last stage the same warps read the accumulators and write the CTA's partial
// The partials of all CTAs are then summed in index order by reduce_splits_2d.
constexpr int WG_THREADS = 320;

struct WgArgs {
    GradSrc dz;
    ValSrc x;
    float* partial;       // [ctas][CO][CI]
    float* gw;            // [CO][CI] (written by the split-sum kernel that follows)
    int* err;
    int P, CO, CI;        // CO, CI: channels one CTA works on (a sub-range of a side that is split over blockIdx.y)
    int COf, CIf;         // the layer's channel counts = row pitches of dy / z and of x, in elements
    int nsa, nsb;         // channel sub-ranges per side; with more than one, the raw rows come by tiled tensor copies
    int pix_per_cta;      // multiple of WSTAGE
    int mtiles, ntiles, NT, tmem_cols;
    int pa, pb;           // 64-channel panels of the two operands per stage (pa even)
    int need_z, R;
    int OPS;              // operand stages: 2, or 1 where the raw ring needs the room
    uint32_t raw_bytes, op_bytes;
};

__global__ void __launch_bounds__(WG_THREADS, 1) pw_wgrad_pipe_kernel(const __grid_constant__ CUtensorMap tm_dy, const __grid_constant__ CUtensorMap tm_z,
                                                                      const __grid_constant__ CUtensorMap tm_x, const WgArgs a) {
    pdl_launch();             // barrier and tensor-memory set-up overlaps the previous kernel; the wait follows it
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2 * MAX_RAW + 5];    // raw_full[R], raw_empty[R], op_full[2], op_empty[2], done
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_store;
    volatile int* abort_flag = &abort_store;
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* sOp = base;                                   // operand stages (a.OPS of them): [A panels][B panels]
    uint8_t* sR = base + (size_t)a.OPS * a.op_bytes;       // raw ring
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int R = a.R;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto raw_full = [&](int s) { return bar0 + 8u * s; };
    auto raw_empty = [&](int s) { return bar0 + 8u * (MAX_RAW + s); };
    auto op_full = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + s); };
    auto op_empty = [&](int s) { return bar0 + 8u * (2 * MAX_RAW + 2 + s); };
    const uint32_t done_bar = bar0 + 8u * (2 * MAX_RAW + 4);
    if (tid == 0) {
        for (int s = 0; s < R; ++s) {
            mbar_init(raw_full(s), 1);
            mbar_init(raw_empty(s), 8);      // one arrival per transform warp
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(op_full(s), 8);
            mbar_init(op_empty(s), 1);
        }
        mbar_init(done_bar, 1);
        abort_store = 0;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), (uint32_t)a.tmem_cols);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    pdl_wait();
    const uint32_t tmem = tmem_slot;
    const int pbeg = blockIdx.x * a.pix_per_cta, pend = min(a.P, pbeg + a.pix_per_cta);
    const int stages = (pend - pbeg + WSTAGE - 1) / WSTAGE;
    const uint32_t rowA = (uint32_t)a.CO * 2u, rowB = (uint32_t)a.CI * 2u;
    const uint32_t offZ = WSTAGE * rowA, offX = offZ * (a.need_z ? 2u : 1u);
    const bool split = a.nsa * a.nsb > 1;
    const int coA = ((int)blockIdx.y % a.nsa) * a.CO, coB = ((int)blockIdx.y / a.nsa) * a.CI;     // first channel of this CTA's sub-ranges

    if (warp == 0) {
        if (lane == 0) {
            const uint8_t* gdy = reinterpret_cast<const uint8_t*>(a.dz.dy);
            const uint8_t* gz = reinterpret_cast<const uint8_t*>(a.dz.z);
            const uint8_t* gx = reinterpret_cast<const uint8_t*>(a.x.p);
            int it = 0;
            for (; it < stages; ++it) {
                const int s = it % R, n = it / R;
                if (n > 0 && !mbar_wait_abortable(raw_empty(s), (uint32_t)((n - 1) & 1), abort_flag)) break;
                const int p0 = pbeg + it * WSTAGE;
                const uint32_t valid = (uint32_t)min(WSTAGE, pend - p0);
                uint8_t* dst = sR + (size_t)s * a.raw_bytes;
                if (split) {
                    // a channel sub-range of 64 pixel rows is not contiguous: one tiled copy per operand lands it as the same
                    // dense rows (a box counts its full size; rows past the last pixel arrive as zeros)
                    mbar_expect_tx(raw_full(s), (uint32_t)WSTAGE * (rowA * (a.need_z ? 2u : 1u) + rowB));
                    tma::load_2d(smem_u32(dst), &tm_dy, coA, p0, raw_full(s));
                    if (a.need_z) tma::load_2d(smem_u32(dst + offZ), &tm_z, coA, p0, raw_full(s));
                    tma::load_2d(smem_u32(dst + offX), &tm_x, coB, p0, raw_full(s));
                    continue;
                }
                mbar_expect_tx(raw_full(s), valid * (rowA * (a.need_z ? 2u : 1u) + rowB));
                bulk_g2s(smem_u32(dst), gdy + (size_t)p0 * rowA, valid * rowA, raw_full(s));
                if (a.need_z) bulk_g2s(smem_u32(dst + offZ), gz + (size_t)p0 * rowA, valid * rowA, raw_full(s));
                bulk_g2s(smem_u32(dst + offX), gx + (size_t)p0 * rowB, valid * rowB, raw_full(s));
            }
            for (int k = (it > R ? it - R : 0); k < it; ++k) mbar_wait(raw_full(k % R), (uint32_t)((k / R) & 1));
        }
    } else if (warp == 1) {
        {
            // every lane runs the loop, the elected lane issues (see the forward / backward-data pipeline)
            const uint32_t leader = elect_leader();
            const uint32_t idesc = make_idesc(a.NT) | (1u << 15) | (1u << 16);
            bool ok = true;
            for (int it = 0; it < stages && ok; ++it) {
                const int st = a.OPS == 2 ? (it & 1) : 0, n = a.OPS == 2 ? (it >> 1) : it;
                if (!mbar_wait_abortable(op_full(st), (uint32_t)(n & 1), abort_flag)) {
                    ok = false;
                    break;
                }
                fence_after_sync();
                const uint32_t a0 = smem_u32(sOp + (size_t)st * a.op_bytes), b0 = a0 + (uint32_t)a.pa * PANEL;
                for (int mt = 0; mt < a.mtiles; ++mt)
                    for (int nt = 0; nt < a.ntiles; ++nt) {
                        const uint32_t d = tmem + (uint32_t)((mt * a.ntiles + nt) * a.NT);
#pragma unroll
                        for (int k = 0; k < WSTAGE / 16; ++k)
                            umma_bf16_lead(d, make_desc_mn(a0 + (uint32_t)mt * 2u * PANEL + k * 2048),
                                           make_desc_mn(b0 + (uint32_t)nt * (uint32_t)(a.NT >> 6) * PANEL + k * 2048), idesc, (it > 0 || k > 0) ? 1u : 0u, leader);
                    }
                umma_commit_lead(op_empty(st), leader);
                __syncwarp();
            }
            if (ok) umma_commit_lead(done_bar, leader);
        }
    } else {
        // ---------------------------------------------------------------- transformers, then epilogue
        // Two uniform passes per stage: every thread first transforms its chunk ja of the dz rows
        // ga, ga + groupsA, ..., then its chunk jb of the x rows gb, gb + groupsB, ...
        const int tix = tid - 64;
        const int ca = a.CO >> 3, cb = a.CI >> 3;
        const int groupsA = 256 / ca, groupsB = 256 / cb;
        const int ja = tix % ca, ga = tix / ca, jb = tix % cb, gb = tix / cb;
        const int rowsA = ga < groupsA ? WSTAGE : 0, rowsB = gb < groupsB ? WSTAGE : 0;
        XfGrad xg;
        XfVal xv;
        xg.init(a.dz, coA + (ja << 3));
        xv.init(a.x, coB + (jb << 3));
        bool ok = true;
        for (int it = 0; it < stages; ++it) {
            const int st = a.OPS == 2 ? (it & 1) : 0, n = a.OPS == 2 ? (it >> 1) : it, s = it % R;
            if (n > 0 && !mbar_wait_abortable(op_empty(st), (uint32_t)((n - 1) & 1), abort_flag)) {
                ok = false;
                break;
            }
            if (!mbar_wait_abortable(raw_full(s), (uint32_t)((it / R) & 1), abort_flag)) {
                ok = false;
                break;
            }
            const uint8_t* raw = sR + (size_t)s * a.raw_bytes;
            uint8_t* dstA = sOp + (size_t)st * a.op_bytes + (uint32_t)(ja >> 3) * PANEL;
            uint8_t* dstB = sOp + (size_t)st * a.op_bytes + (uint32_t)(a.pa + (jb >> 3)) * PANEL;
            const int valid = min(WSTAGE, pend - (pbeg + it * WSTAGE));
            // straight-line bodies: rows past the end of the CTA's range are transformed like any
            // other (stale but in-bounds shared memory) and zeroed afterwards
#pragma unroll 1
            for (int kr = ga; kr < rowsA; kr += groupsA) {
                const uint4 r0 = *reinterpret_cast<const uint4*>(raw + (size_t)kr * rowA + (ja << 4));
                uint4 q4 = a.need_z ? xg.apply(r0, *reinterpret_cast<const uint4*>(raw + offZ + (size_t)kr * rowA + (ja << 4))) : r0;
                if (kr >= valid) q4 = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(dstA + kr * 128 + (((ja & 7) ^ (kr & 7)) << 4)) = q4;
            }
#pragma unroll 1
            for (int kr = gb; kr < rowsB; kr += groupsB) {
                uint4 q4 = xv.apply(*reinterpret_cast<const uint4*>(raw + offX + (size_t)kr * rowB + (jb << 4)));
                if (kr >= valid) q4 = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(dstB + kr * 128 + (((jb & 7) ^ (kr & 7)) << 4)) = q4;
            }
            // one arrival per warp (an arrival is a shared-memory atomic: hundreds of them per hand-off serialise)
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(raw_empty(s));
                mbar_arrive(op_full(st));
            }
        }
        if (ok && stages > 0) ok = mbar_wait_abortable(done_bar, 0u, abort_flag);
        if (ok) {
            fence_after_sync();
            const int q = warp & 3, half = (warp - 2) >> 2;    // two warps share each lane quarter
            float* pbase = a.partial + (size_t)blockIdx.x * a.COf * a.CIf + (size_t)coA * a.CIf + coB;
            for (int mt = 0; mt < a.mtiles; ++mt) {
                const int k = mt * TM + q * 32 + lane;
                for (int nt = 0; nt < a.ntiles; ++nt)
                    for (int g = half; g < (a.NT >> 4); g += 2) {
                        float v[16];
                        if (stages > 0) {
                            tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((mt * a.ntiles + nt) * a.NT + (g << 4)), v);
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = 0.f;
                        }
                        const int c = nt * a.NT + (g << 4);
                        if (k < a.CO) {
#pragma unroll
                            for (int hh = 0; hh < 4; ++hh)
                                if (c + hh * 4 < a.CI)
                                    *reinterpret_cast<float4*>(pbase + (size_t)k * a.CIf + c + hh * 4) = make_float4(v[hh * 4], v[hh * 4 + 1], v[hh * 4 + 2], v[hh * 4 + 3]);
                        }
                    }
            }
        }
    }
    fence_before_sync();
    __syncthreads();
    if (tid == 0 && abort_store) atomicExch(a.err, 1);
    if (warp == 1) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
}

// out[i] = sum_k partial[k][i], k in index order.  A block of 1024 threads owns 32 outputs:
// thread (kg, il) adds the partials kg, kg+32, ... of output il (32 consecutive outputs per
// load: coalesced; all of a thread's loads are issued before the additions), the 32 sub-sums
// are combined in fixed order through shared memory.
__global__ void __launch_bounds__(1024) reduce_splits_2d(const float* __restrict__ partial, int splits, size_t n, float* __restrict__ out) {
    pdl_wait();
    pdl_launch();
    __shared__ float sh[32][33];
    const int il = threadIdx.x & 31, kg = threadIdx.x >> 5;
    const size_t i = (size_t)blockIdx.x * 32 + il;
    float acc = 0.f;
    if (i < n) {
        for (int k0 = kg; k0 < splits; k0 += 32 * 8) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = (k0 + 32 * u < splits) ? partial[(size_t)(k0 + 32 * u) * n + i] : 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) acc += v[u];
        }
    }
    sh[kg][il] = acc;
    __syncthreads();
    if (kg == 0 && i < n) {
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < 32; ++k) s += sh[k][il];
        out[i] = s;
    }
}

// Plans the kernel for a.nsa x a.nsb channel sub-ranges of the layer's a.COf x a.CIf weight gradient.
bool plan_wgrad(WgArgs& a, size_t* smem, size_t scratch_floats, int n_sm) {
    if (a.COf % a.nsa || a.CIf % a.nsb) return false;
    a.CO = a.COf / a.nsa;
    a.CI = a.CIf / a.nsb;
    const int ns = a.nsa * a.nsb;
    if (ns > 1 && (a.CO % 64 || a.CI % 64 || a.CO > 256 || a.CI > 256)) return false;     // box of a tiled copy: at most 256 elements wide
    if (a.CO > 512 || a.CI > 512 || (a.CO + a.CI) / 8 > 256) return false;
    a.ntiles = (a.CI + 255) / 256;
    a.NT = ((a.CI + a.ntiles - 1) / a.ntiles + 63) / 64 * 64;      // whole panels per N tile
    if (a.ntiles == 1) a.NT = (a.CI + 15) / 16 * 16;
    a.mtiles = (a.CO + TM - 1) / TM;
    int cols = a.mtiles * a.ntiles * a.NT;
    a.tmem_cols = 32;
    while (a.tmem_cols < cols) a.tmem_cols <<= 1;
    if (a.tmem_cols > 512) return false;
    a.pa = a.mtiles * 2;
    a.pb = a.ntiles == 1 ? (a.NT + 63) / 64 : a.ntiles * (a.NT / 64);
    a.op_bytes = (uint32_t)(a.pa + a.pb) * PANEL;
    size_t rb = (size_t)WSTAGE * (a.CO * 2 * (a.need_z ? 2 : 1) + a.CI * 2);
    rb = (rb + 127) / 128 * 128;
    a.raw_bytes = (uint32_t)rb;
    const size_t budget = 226 * 1024 - 1024;
    a.OPS = 2 * (size_t)a.op_bytes + 2 * rb <= budget ? 2 : 1;
    const size_t fixed = (size_t)a.OPS * a.op_bytes;
    if (fixed + 2 * rb > budget) return false;
    size_t r = (budget - fixed) / rb;
    if (r > 4) r = 4;
    a.R = (int)r;
    *smem = fixed + r * rb + 1024;
    size_t out_elems = (size_t)a.COf * a.CIf;
    int ctas = n_sm / ns;                       // pixel ranges; every range is worked on by one CTA per pair of sub-ranges
    int max_by_pix = (a.P + 2 * WSTAGE - 1) / (2 * WSTAGE);
    if (ctas > max_by_pix) ctas = max_by_pix;
    size_t cap = scratch_floats / out_elems;
    if ((size_t)ctas > cap) ctas = (int)cap;
    if (ctas < 1) return false;
    int ppc = (a.P + ctas - 1) / ctas;
    ppc = (ppc + WSTAGE - 1) / WSTAGE * WSTAGE;
    a.pix_per_cta = ppc;
    return true;
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
    // One tile per CTA, so the phases of a tile (load, multiply, store) overlap only across the CTAs of an SM: keep the
    // staged reduction chunk small enough for three of them (or as many as the tensor-memory columns allow).
    const int want = 512 / t.tmem_cols < 3 ? 512 / t.tmem_cols : 3;
    while (t.KC > KB && ((size_t)(t.KC / KB) * (TM + t.NT) * 128 + 1024) * want > 220 * 1024) t.KC >>= 1;
    t.KC = (t.KC + KB - 1) / KB * KB;
    t.smem = (size_t)(t.KC / KB) * (TM + t.NT) * 128 + 1024;
    return t;
}

template <bool BWD> void launch(const PwArgs& a0, const Tiling& t, int kind, double bytes, cudaStream_t st) {
    PwArgs a = a0;
    a.NT = t.NT; a.KC = t.KC; a.tmem_cols = t.tmem_cols;
    smem_limit_once<103 + (BWD ? 50 : 0)>(pw_tc_kernel<BWD>, 200 * 1024);
    LaunchScope ls(kind, bytes, 2.0 * a.P * a.N * a.K, st);
    dim3 grid((a.P + TM - 1) / TM, t.ntiles);
    launch_pdl(pw_tc_kernel<BWD>, grid, NTHREADS, t.smem, st, a);
}

}  // namespace

bool pw_tc_supported(int dtype, const ConvGeom& g, bool bwd_data) {
    (void)bwd_data;
    return dtype == 1 && g.k == 1 && g.pad == 0 && g.ci % 8 == 0 && g.co % 8 == 0 && g.ci >= 8 && g.co >= 8;
}

int pw_fwd_tc(const ConvGeom& g, const ValSrc& x, const __nv_bfloat16* wb, const float* bias, void* z, const float* pivot, float* partial,
              size_t partial_floats, int* err, cudaStream_t st) {
    PwArgs a{};
    a.x = x; a.w = wb; a.bias = bias; a.out = (__nv_bfloat16*)z; a.err = err;
    a.P = g.n * g.ho * g.wo; a.K = g.ci; a.N = g.co;
    a.stride = g.stride; a.ho = g.ho; a.wo = g.wo; a.hi = g.hi; a.wi = g.wi;
    double bytes = 2.0 * ((double)a.P * a.K + (double)a.P * a.N) + 2.0 * a.N * a.K;
    if (g.stride == 1) {
        PipeArgs pa{};
        pa.x = x; pa.w = wb; pa.bias = bias; pa.out = (__nv_bfloat16*)z; pa.err = err;
        pa.P = a.P; pa.K = a.K; pa.N = a.N; pa.tiles = (a.P + TM - 1) / TM; pa.need_z = 0;
        if (pivot && partial) {
            pa.pivot = pivot;
            pa.stat_partial = partial;
        }
        size_t smem = 0;
        alignas(64) CUtensorMap tm_out;
        if (plan_pipe(pa, &smem) && make_out_map(z, pa.P, pa.N, &tm_out)) return launch_pipe<false>(pa, tm_out, smem, K_PW_FWD_TC, bytes, partial_floats, st);
    }
    // more than 256 channels on a side: the streaming kernel, where the layer fits it
    if (g.stride == 1 && !bias && pw_stream(false, a.P, a.K, a.N, x, GradSrc{}, wb, nullptr, z, err, K_PW_FWD_TC, bytes, st)) return 0;
    Tiling t = pick_tiling(a.K, a.N);
    launch<false>(a, t, K_PW_FWD_TC, bytes, st);
    return 0;
}

int pw_bwd_data_tc(const ConvGeom& g, const GradSrc& dz, const __nv_bfloat16* wtb, const void* addend, void* dx, const BnRed* red, int* err,
                   cudaStream_t st) {
    PwArgs a{};
    a.dz = dz; a.w = wtb; a.addend = addend; a.out = (__nv_bfloat16*)dx; a.err = err;
    a.P = g.n * g.ho * g.wo; a.K = g.co; a.N = g.ci;
    a.stride = g.stride; a.ho = g.ho; a.wo = g.wo; a.hi = g.hi; a.wi = g.wi;
    double bytes = 2.0 * (double)a.P * a.K * ((dz.act != ACT_NONE || dz.k1) ? 2.0 : 1.0) + 2.0 * (double)a.P * a.N * (addend ? 2.0 : 1.0) +
                   2.0 * a.N * a.K;
    if (g.stride > 1) {
        // only the sampled pixels receive a term: the rest of dx is the addend (or zero); the kernel
        // then accumulates in place at the sampled positions
        const size_t full = (size_t)g.n * g.hi * g.wi * g.ci * 2;
        if (!addend) cudaMemsetAsync(dx, 0, full, st);
        else if (addend != dx) cudaMemcpyAsync(dx, addend, full, cudaMemcpyDeviceToDevice, st);
        a.addend = dx;
        Tiling t = pick_tiling(a.K, a.N);
        launch<true>(a, t, K_PW_BWD_DATA_TC, bytes + (double)full, st);
        return 0;
    }
    for (int with_red = red ? 1 : 0; with_red >= 0; --with_red) {
        PipeArgs pa{};
        pa.dz = dz; pa.w = wtb; pa.addend = addend; pa.out = (__nv_bfloat16*)dx; pa.err = err;
        pa.P = a.P; pa.K = a.K; pa.N = a.N; pa.tiles = (a.P + TM - 1) / TM; pa.need_z = (dz.act != ACT_NONE || dz.k1) ? 1 : 0;
        if (with_red) {
            pa.rz = (const __nv_bfloat16*)red->z;
            pa.r_scale = red->scale; pa.r_shift = red->shift; pa.r_mean = red->mean; pa.r_rstd = red->rstd;
            pa.r_act = red->act;
            pa.r_partial = red->partial;
        }
        size_t smem = 0;
        alignas(64) CUtensorMap tm_out;
        if (plan_pipe(pa, &smem) && make_out_map(dx, pa.P, pa.N, &tm_out))
            return launch_pipe<true>(pa, tm_out, smem, K_PW_BWD_DATA_TC, bytes, with_red ? red->partial_floats : 0, st);
    }
    // the streaming kernel where the gradient needs no transform: with one, its 64-channel blocks are too small a unit of
    // work for the transform warps' hand-offs and the one-tile kernel below is as fast
    if (!grad_needs_z(dz) && pw_stream(true, a.P, a.K, a.N, ValSrc{}, dz, wtb, addend, dx, err, K_PW_BWD_DATA_TC, bytes, st)) return 0;
    Tiling t = pick_tiling(a.K, a.N);
    launch<true>(a, t, K_PW_BWD_DATA_TC, bytes, st);
    return 0;
}

void pw_bwd_weight_tc(const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw, int* err,
                      cudaStream_t st) {
    if (g.stride == 1) {
        smem_limit_once<104>(pw_wgrad_pipe_kernel, 226 * 1024);
        const int n_sm = sm_count();
        WgArgs wa{};
        wa.dz = dz; wa.x = x; wa.partial = scratch; wa.gw = gw; wa.err = err;
        wa.P = g.n * g.ho * g.wo; wa.COf = g.co; wa.CIf = g.ci;
        wa.need_z = (dz.act != ACT_NONE || dz.k1) ? 1 : 0;
        size_t smem = 0;
        // the whole gradient in one CTA's tensor memory where its stages fit; else the wider side in 2 or 4 channel sub-ranges
        // (the other side's rows are then read once per sub-range, by CTAs that run side by side: a re-read from L2)
        static const int kSplits[3][2] = {{1, 1}, {4, 1}, {2, 1}};
        bool planned = false;
        for (int i = 0; i < 3 && !planned; ++i) {
            wa.nsa = g.co >= g.ci ? kSplits[i][0] : kSplits[i][1];
            wa.nsb = g.co >= g.ci ? kSplits[i][1] : kSplits[i][0];
            planned = plan_wgrad(wa, &smem, scratch_floats, n_sm);
        }
        alignas(64) CUtensorMap tm_dy, tm_z, tm_x;
        memset(&tm_dy, 0, sizeof(tm_dy)); memset(&tm_z, 0, sizeof(tm_z)); memset(&tm_x, 0, sizeof(tm_x));
        if (planned && wa.nsa * wa.nsb > 1) {
            const uint64_t da[2] = {(uint64_t)wa.COf, (uint64_t)wa.P}, db[2] = {(uint64_t)wa.CIf, (uint64_t)wa.P};
            const uint64_t sa[1] = {(uint64_t)wa.COf * 2}, sb[1] = {(uint64_t)wa.CIf * 2};
            const uint32_t ba[2] = {(uint32_t)wa.CO, (uint32_t)WSTAGE}, bb[2] = {(uint32_t)wa.CI, (uint32_t)WSTAGE};
            planned = tma::encode_bf16(&tm_dy, dz.dy, 2, da, sa, ba, false) && (!wa.need_z || tma::encode_bf16(&tm_z, dz.z, 2, da, sa, ba, false)) &&
                      tma::encode_bf16(&tm_x, x.p, 2, db, sb, bb, false);
        }
        if (planned) {
            int ctas = (wa.P + wa.pix_per_cta - 1) / wa.pix_per_cta;
            double bytes = 2.0 * (double)wa.P * wa.COf * (wa.need_z ? 2.0 : 1.0) + 2.0 * (double)wa.P * wa.CIf + 4.0 * wa.COf * wa.CIf;   // operands and gradient once: partials belong to the split sum
            {
                LaunchScope ls(K_PW_BWD_WEIGHT_TC, bytes, 2.0 * wa.P * wa.COf * wa.CIf, st);
                launch_pdl(pw_wgrad_pipe_kernel, dim3(ctas, wa.nsa * wa.nsb), WG_THREADS, smem, st, tm_dy, tm_z, tm_x, wa);
            }
            size_t out_elems = (size_t)wa.COf * wa.CIf;
            LaunchScope ls(K_REDUCE_SPLITS, 4.0 * out_elems * (ctas + 1), (double)out_elems * ctas, st);
            if (out_elems % 4 == 0 && (reinterpret_cast<uintptr_t>(scratch) | reinterpret_cast<uintptr_t>(gw)) % 16 == 0)
                reduce_splits_f4(scratch, ctas, out_elems, gw, st);
            else
                launch_pdl(reduce_splits_2d, (unsigned)((out_elems + 31) / 32), 1024, 0, st, scratch, ctas, out_elems, gw);
            return;
        }
    }
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
    int splits = (2 * sm_count() + mtiles * ntiles - 1) / (mtiles * ntiles);
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
    smem_limit_once<105>(pw_bwd_weight_tc_kernel, 200 * 1024);
    double bytes = 2.0 * (double)a.P * a.CO * ((dz.act != ACT_NONE || dz.k1) ? 2.0 : 1.0) + 2.0 * (double)g.n * g.hi * g.wi * a.CI +
                   4.0 * out_elems;
    {
        LaunchScope ls(K_PW_BWD_WEIGHT_TC, bytes, 2.0 * a.P * a.CO * a.CI, st);
        launch_pdl(pw_bwd_weight_tc_kernel, dim3(mtiles, splits, ntiles), NTHREADS, smem, st, a);
    }
    LaunchScope ls(K_REDUCE_SPLITS, 4.0 * out_elems * (splits + 1), (double)out_elems * splits, st);
    launch_pdl(reduce_splits_tc, (unsigned)((out_elems + 255) / 256), 256, 0, st, scratch, splits, out_elems, gw);
}

}  // namespace ast
