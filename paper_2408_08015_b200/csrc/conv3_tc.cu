// Dense 3x3 convolution (stride 1, pad 1) as an implicit GEMM on tcgen05: forward and
// backward-data.
//
// Pixels of one image are addressed in *padded, flattened* coordinates f = hp*(W+2) + wp.  In
// these coordinates tap (r,s) of output position f reads position f + (r-1)*(W+2) + (s-1): a
// constant row offset.  A CTA owns 128 consecutive positions; it stages the 128 + 2(W+2) + 2
// positions they touch ONCE (producer BatchNorm + activation, or the BatchNorm-backward
// transform, applied on the way; padding positions are zeros) as K-major rows of 64 channels,
// and every tap's A operand is the same buffer seen through a descriptor whose start address is
// moved by the tap's row offset.  Per tap the weights [N][C] are streamed into one of two
// shared-memory stages while the previous tap's MMAs run; the 9*C/16 MMAs accumulate into one
// tensor-memory tile.  Positions that are padding produce values that are never stored.
#include <cuda_bf16.h>

#include "kernels.h"
#include "tc_common.cuh"

namespace ast {
namespace {

using namespace tc;
constexpr int C3_THREADS = 256;

struct C3Args {
    ValSrc x;                  // forward operand
    GradSrc dz;                // backward operand
    const __nv_bfloat16* w;    // forward: [N][9][C] (N = c_out, C = c_in); backward: [N][9][C] with N = c_in, C = c_out
    const void* addend;        // backward only, may be null
    __nv_bfloat16* out;        // [n][H][W][N]
    int* err;
    int n_img, H, W, C, N;     // C: reduction channels (multiple of 64), N: output channels (multiple of 16, <= 256)
    int tiles_per_img, rows_pad, tmem_cols;
    int flip;                  // backward: tap t uses weight tap 8 - t
    int resident;              // all nine taps' weights fit in shared memory beside the staged rows: loaded once, before the
                               // dependency wait, and the 9 * C/16 MMAs are issued back to back
};

// K-major, 128-byte swizzle, start address anywhere on a 128-byte row of a 1024-byte aligned
// buffer.  The swizzle is a function of the shared-memory address bits (16-byte chunk index XOR
// address bits 7..9), and the rows were written with the same function of their address, so a
// start address moved by whole rows needs no correction: the base-offset field stays 0.
__device__ __forceinline__ uint64_t make_desc_row(uint32_t smem_addr) { return make_desc(smem_addr); }

template <bool BWD> __global__ void __launch_bounds__(C3_THREADS) conv3_tc_kernel(const C3Args a) {
    // barriers, tensor memory and (resident form) the weights, which only the refresh kernel writes, are set up before
    // the dependency wait and overlap the previous kernel's tail
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2];
    __shared__ uint32_t tmem_slot;
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Wp = a.W + 2;
    const int kbs = a.C >> 6;                               // 64-channel blocks
    const uint32_t a_block = (uint32_t)a.rows_pad * 128u;   // bytes of one channel block of the staged rows
    const uint32_t b_stage = (uint32_t)kbs * (uint32_t)a.N * 128u;
    uint8_t* sA = base;
    uint8_t* sB = base + (size_t)kbs * a_block;
    const int img = blockIdx.x / a.tiles_per_img, tile = blockIdx.x - img * a.tiles_per_img;
    const int f0 = Wp + 1 + tile * TM;                      // first output position of this CTA
    const int fs0 = f0 - Wp - 1;                            // first staged position
    const int rows = TM + 2 * Wp + 2;
    const uint32_t bar0 = smem_u32(&bars[0]), bar1 = smem_u32(&bars[1]);

    if (tid == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar1, 1);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), (uint32_t)a.tmem_cols);
        tmem_relinquish();
    }
    if (a.resident) {
        const int vprw = a.C >> 3;
#pragma unroll 4
        for (int v = tid; v < 9 * a.N * vprw; v += C3_THREADS) {
            const int t = v / (a.N * vprw), rem = v - t * (a.N * vprw);
            const int n = rem / vprw, j = rem - n * vprw;
            const int wt = a.flip ? 8 - t : t;
            uint4 q = __ldg(reinterpret_cast<const uint4*>(a.w + ((size_t)n * 9 + wt) * a.C) + j);
            *reinterpret_cast<uint4*>(sB + (size_t)t * b_stage + tile_off(n, j, a.N)) = q;
        }
    }
    pdl_wait();
    // ---- stage the input rows once: position -> (hp, wp); interior positions are pixels ----
    // A thread owns one 16-byte channel chunk (its transform coefficients stay in registers) and every (256 / chunks)-th
    // row; the global loads of four rows are issued together before any of them is transformed, so that their
    // latencies overlap instead of adding up.
    {
        const int vpr = a.C >> 3;                       // 8 or a multiple of 8 dividing 256
        const int j = tid % vpr, step = C3_THREADS / vpr;
        const int c0 = j << 3;
        const bool need_z = BWD && (a.dz.act != ACT_NONE || a.dz.k1 != nullptr);
        XfVal xv;
        XfGrad xg;
        if (BWD) xg.init(a.dz, c0);
        else xv.init(a.x, c0);
        const uint4* src = reinterpret_cast<const uint4*>(BWD ? a.dz.dy : a.x.p);
        const uint4* srcz = reinterpret_cast<const uint4*>(a.dz.z);
        constexpr int U = 4;
        for (int rb = tid / vpr; rb < rows; rb += U * step) {
            uint4 raw[U], rawz[U];
            bool ok[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = rb + u * step;
                const int f = fs0 + r;
                const int hp = f / Wp, wp = f - hp * Wp;
                ok[u] = r < rows && f >= 0 && hp >= 1 && hp <= a.H && wp >= 1 && wp <= a.W;
                raw[u] = rawz[u] = make_uint4(0, 0, 0, 0);
                if (ok[u]) {
                    const size_t e = ((((size_t)img * a.H + (hp - 1)) * a.W + (wp - 1)) * a.C + c0) >> 3;
                    raw[u] = __ldg(src + e);
                    if (need_z) rawz[u] = __ldg(srcz + e);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int r = rb + u * step;
                if (r < rows) {
                    uint4 q = make_uint4(0, 0, 0, 0);
                    if (ok[u]) q = BWD ? (need_z ? xg.apply(raw[u], rawz[u]) : raw[u]) : xv.apply(raw[u]);
                    *reinterpret_cast<uint4*>(sA + (size_t)(j >> 3) * a_block + (size_t)r * 128 + ((((uint32_t)j & 7u) ^ ((uint32_t)r & 7u)) << 4)) = q;
                }
            }
        }
    }
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = tmem_slot;
    const uint32_t idesc = make_idesc(a.N);

    // ---- nine taps: stream the tap's weights into stage t&1, then its C/16 MMAs ----
    uint32_t ph[2] = {0, 0};
    bool bad = false;
    const int vpr = a.C >> 3;
    if (a.resident) {
        if (tid == 0) {
            for (int t = 0; t < 9; ++t) {
                const int r = t / 3, s = t - r * 3;
                const uint32_t a0 = smem_u32(sA) + (uint32_t)(r * Wp + s) * 128u;
                const uint32_t b0 = smem_u32(sB) + (uint32_t)t * b_stage;
                for (int k = 0; k < (a.C >> 4); ++k) {
                    const int kb = k >> 2, ks = k & 3;
                    umma_bf16(tmem, make_desc_row(a0 + (uint32_t)kb * a_block + (uint32_t)ks * 32u),
                              make_desc(b0 + (uint32_t)kb * (uint32_t)a.N * 128u + (uint32_t)ks * 32u), idesc, (t > 0 || k > 0) ? 1u : 0u);
                }
            }
            umma_commit(bar0);
        }
    }
    for (int t = 0; t < 9 && !a.resident; ++t) {
        const int st = t & 1;
        if (t >= 2) {                                   // the MMAs of tap t-2 read this weight stage
            bool ok = mbar_wait(st ? bar1 : bar0, ph[st]);
            ph[st] ^= 1;
            if (!__syncthreads_and(ok ? 1 : 0)) {
                bad = true;
                break;
            }
        }
        const int wt = a.flip ? 8 - t : t;
        uint8_t* dstB = sB + (size_t)st * b_stage;
#pragma unroll 4
        for (int v = tid; v < a.N * vpr; v += C3_THREADS) {
            const int n = v / vpr, j = v - n * vpr;
            uint4 q = __ldg(reinterpret_cast<const uint4*>(a.w + ((size_t)n * 9 + wt) * a.C) + j);
            *reinterpret_cast<uint4*>(dstB + tile_off(n, j, a.N)) = q;
        }
        fence_async_smem();
        __syncthreads();
        if (tid == 0) {
            fence_after_sync();
            const int r = t / 3, s = t - r * 3;
            const uint32_t a0 = smem_u32(sA) + (uint32_t)(r * Wp + s) * 128u;
            const uint32_t b0 = smem_u32(dstB);
            for (int k = 0; k < (a.C >> 4); ++k) {
                const int kb = k >> 2, ks = k & 3;
                umma_bf16(tmem, make_desc_row(a0 + (uint32_t)kb * a_block + (uint32_t)ks * 32u),
                          make_desc(b0 + (uint32_t)kb * (uint32_t)a.N * 128u + (uint32_t)ks * 32u), idesc, (t > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(st ? bar1 : bar0);
        }
    }
    if (!bad) {                                         // the last commit (tap 8, stage 0) covers every MMA
        bool ok = mbar_wait(bar0, ph[0]);
        if (!__syncthreads_and(ok ? 1 : 0)) bad = true;
    }
    fence_after_sync();
    __syncthreads();
    if (bad) {
        if (tid == 0) atomicExch(a.err, 1);
    } else {
        const int q = warp & 3, half = warp >> 2;
        const int f = f0 + q * 32 + lane;
        const int hp = f / Wp, wp = f - hp * Wp;
        const bool pix = hp >= 1 && hp <= a.H && wp >= 1 && wp <= a.W;
        const size_t e0 = (((size_t)img * a.H + (hp - 1)) * a.W + (wp - 1)) * a.N;
        for (int g = half; g < (a.N >> 4); g += 2) {
            float v[16];
            tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g << 4), v);
            if (pix) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    float* vv = v + (hh << 3);
                    const size_t e = e0 + (g << 4) + (hh << 3);
                    if (BWD && a.addend) {
                        float ad[8];
                        Vec<__nv_bfloat16> av;
                        av.load(a.addend, e >> 3);
                        av.unpack(ad);
#pragma unroll
                        for (int i = 0; i < 8; ++i) vv[i] += ad[i];
                    }
                    *reinterpret_cast<uint4*>(a.out + e) = pack8(vv);
                }
            }
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
}

// ---------------------------------------------------------------------------------------------
// Persistent form of the same implicit GEMM for layers of up to 128 reduction channels on maps up to 61 pixels wide
// (every dense 3x3 layer of the ResNet stage).  One CTA per SM walks over tiles and keeps resident, for all nine
// taps, the weights of the 64 output channels it owns (wider layers are split over CTAs by output channel), so that
// per tile only the halo rows are brought in.  The loop is software-pipelined with all threads in the same role:
//
//   iteration i:  transform the prefetched raw rows of tile i into the operand buffer -> issue its 9*C/16 MMAs into
//                 accumulator i&1 -> issue the global loads of tile i+1's rows into registers -> wait for the MMAs of
//                 tile i-1 and store its accumulator (i-1)&1
//
// so the MMAs of a tile run while the next tile's loads are in flight and the previous tile is being stored.  With 64
// reduction channels two operand buffers fit and the transform of tile i+1 overlaps the MMAs of tile i as well.
constexpr int C3P_NH = 64;             // output channels per CTA

struct C3PArgs {
    ValSrc x;
    GradSrc dz;
    const __nv_bfloat16* w;    // [N][9][C]
    const void* addend;
    __nv_bfloat16* out;        // [n][H][W][N]
    int* err;
    int n_img, H, W, C, N;
    int tiles_per_img, total_tiles, rows_pad, n_split, nbuf, flip;
};

// NTHR = 512 with one CTA per SM (128 reduction channels: the resident weights take 147 KB), or 256 with two CTAs per SM (64
// channels: 74 KB of weights and a 31 KB operand buffer each), which then overlap each other's load and barrier waits.
template <bool BWD, int IT, int NTHR> __global__ void __launch_bounds__(NTHR, NTHR == 256 ? 2 : 1) conv3_persist_kernel(const C3PArgs a) {
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2];
    __shared__ uint32_t tmem_slot;
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Wp = a.W + 2;
    const int kbs = a.C >> 6;
    const uint32_t a_block = (uint32_t)a.rows_pad * 128u;
    const uint32_t a_buf = (uint32_t)kbs * a_block;
    const uint32_t b_tap = (uint32_t)kbs * C3P_NH * 128u;
    uint8_t* sA = base;
    uint8_t* sB = base + (size_t)a.nbuf * a_buf;
    const int half = blockIdx.x % a.n_split, n0 = half * C3P_NH;
    const int cta = blockIdx.x / a.n_split, nctas = gridDim.x / a.n_split;
    const int rows = TM + 2 * Wp + 2;
    const uint32_t bar[2] = {smem_u32(&bars[0]), smem_u32(&bars[1])};
    if (tid == 0) {
        mbar_init(bar[0], 1);
        mbar_init(bar[1], 1);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 2 * C3P_NH);
        tmem_relinquish();
    }
    // resident weights of this CTA's 64 output channels, all nine taps (written only by the refresh kernel, which never
    // releases its dependents early: safe to read before the dependency wait)
    {
        const int vprw = a.C >> 3;
#pragma unroll 4
        for (int v = tid; v < 9 * C3P_NH * vprw; v += NTHR) {
            const int t = v / (C3P_NH * vprw), rem = v - t * (C3P_NH * vprw);
            const int n = rem / vprw, j = rem - n * vprw;
            const int wt = a.flip ? 8 - t : t;
            const uint4 q = __ldg(reinterpret_cast<const uint4*>(a.w + ((size_t)(n0 + n) * 9 + wt) * a.C) + j);
            *reinterpret_cast<uint4*>(sB + (size_t)t * b_tap + tile_off(n, j, C3P_NH)) = q;
        }
    }
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    pdl_wait();
    const uint32_t tmem = tmem_slot;
    const uint32_t idesc = make_idesc(C3P_NH);

    // staging role: one 16-byte channel chunk (coefficients in registers), every (512 / chunks)-th row
    const int vpr = a.C >> 3;
    const int j = tid % vpr, step = NTHR / vpr, r_first = tid / vpr;
    const int c0 = j << 3;
    const bool need_z = BWD && grad_needs_z(a.dz);
    XfVal xv;
    XfGrad xg;
    if (BWD) xg.init(a.dz, c0);
    else xv.init(a.x, c0);
    const uint4* src = reinterpret_cast<const uint4*>(BWD ? a.dz.dy : a.x.p);
    const uint4* srcz = reinterpret_cast<const uint4*>(a.dz.z);
    uint4 raw[IT], rawz[IT];
    uint32_t okmask = 0;

    // Positions advance by `step` rows per item: (hp, wp) of a row follow from the previous row's by additions, so that a
    // tile costs one integer division per thread; element indices stay in 32 bits, in units of 16-byte vectors.
    const int step_q = step / Wp, step_r = step - step_q * Wp;
    const uint32_t W_u = (uint32_t)a.W, H_u = (uint32_t)a.H;
    auto prefetch = [&](int tl) {
        const int img = tl / a.tiles_per_img, tile = tl - img * a.tiles_per_img;
        const int f0 = tile * TM + r_first;                 // first staged position of this thread (first output position - Wp - 1)
        int hp = f0 / Wp, wp = f0 - hp * Wp;
        const uint32_t img_row0 = (uint32_t)img * H_u;
        okmask = 0;
#pragma unroll
        for (int u = 0; u < IT; ++u) {
            const bool ok = r_first + u * step < rows && (uint32_t)(hp - 1) < H_u && (uint32_t)(wp - 1) < W_u;
            raw[u] = make_uint4(0, 0, 0, 0);
            if (BWD) rawz[u] = make_uint4(0, 0, 0, 0);
            if (ok) {
                const uint32_t e = ((img_row0 + (uint32_t)(hp - 1)) * W_u + (uint32_t)(wp - 1)) * (uint32_t)vpr + (uint32_t)j;
                raw[u] = __ldg(src + e);
                if (need_z) rawz[u] = __ldg(srcz + e);
                okmask |= 1u << u;
            }
            wp += step_r;
            hp += step_q;
            if (wp >= Wp) {
                wp -= Wp;
                ++hp;
            }
        }
    };
    auto store_stage = [&](int buf) {
        uint8_t* dst = sA + (size_t)buf * a_buf + (size_t)(j >> 3) * a_block;
#pragma unroll
        for (int u = 0; u < IT; ++u) {
            const int r = r_first + u * step;
            if (r < rows) {
                uint4 q = make_uint4(0, 0, 0, 0);
                if (okmask & (1u << u)) q = BWD ? (need_z ? xg.apply(raw[u], rawz[u]) : raw[u]) : xv.apply(raw[u]);
                *reinterpret_cast<uint4*>(dst + (size_t)r * 128 + ((((uint32_t)j & 7u) ^ ((uint32_t)r & 7u)) << 4)) = q;
            }
        }
    };
    auto issue = [&](int buf, int acc) {
        const uint32_t abase = smem_u32(sA) + (uint32_t)buf * a_buf, bbase = smem_u32(sB);
        const uint32_t d = tmem + (uint32_t)(acc * C3P_NH);
        // descriptor = constant fields + (address >> 4): all addresses here are 16-byte multiples below 256 KB
        const uint64_t dconst = make_desc(0);
#pragma unroll
        for (int t = 0; t < 9; ++t) {
            const int r = t / 3, s = t - r * 3;
            const uint32_t a0 = (abase + (uint32_t)(r * Wp + s) * 128u) >> 4;
            const uint32_t b0 = (bbase + (uint32_t)t * b_tap) >> 4;
            for (int kb = 0; kb < kbs; ++kb) {
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16(d, dconst + (uint64_t)(a0 + (((uint32_t)kb * a_block + (uint32_t)ks * 32u) >> 4)),
                              dconst + (uint64_t)(b0 + (((uint32_t)kb * C3P_NH * 128u + (uint32_t)ks * 32u) >> 4)), idesc, (t > 0 || kb > 0 || ks > 0) ? 1u : 0u);
            }
        }
        umma_commit(bar[acc]);
    };
    // warp & 3 = tensor-memory lane quarter (32 positions), warp >> 2 = which share of the 64 output channels (16 or 32 of them)
    auto epilogue = [&](int tl, int acc) {
        const int img = tl / a.tiles_per_img, tile = tl - img * a.tiles_per_img;
        const int q = warp & 3;
        const int f = Wp + 1 + tile * TM + q * 32 + lane;
        const int hp = f / Wp, wp = f - hp * Wp;
        const bool pix = hp >= 1 && hp <= a.H && wp >= 1 && wp <= a.W;
        constexpr int CHUNKS = C3P_NH / 16 / (NTHR / 128);       // 16-column chunks per warp
#pragma unroll
        for (int ch = 0; ch < CHUNKS; ++ch) {
        const int cg = (warp >> 2) * CHUNKS + ch;
        float v[16];
        tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * C3P_NH + (cg << 4)), v);
        if (pix) {
            const size_t e0 = (((size_t)img * a.H + (hp - 1)) * a.W + (wp - 1)) * a.N + n0 + (cg << 4);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                float* vv = v + (hh << 3);
                const size_t e = e0 + (hh << 3);
                if (BWD && a.addend) {
                    float ad[8];
                    Vec<__nv_bfloat16> av;
                    av.load(a.addend, e >> 3);
                    av.unpack(ad);
#pragma unroll
                    for (int i = 0; i < 8; ++i) vv[i] += ad[i];
                }
                *reinterpret_cast<uint4*>(a.out + e) = pack8(vv);
            }
        }
        }
    };

    const int my = cta < a.total_tiles ? (a.total_tiles - cta + nctas - 1) / nctas : 0;
    uint32_t ph[2] = {0, 0};
    bool bad = false;
    auto wait_mma = [&](int i) -> bool {       // block-uniform result
        const int acc = i & 1;
        const bool ok = mbar_wait(bar[acc], ph[acc]);
        ph[acc] ^= 1;
        return __syncthreads_and(ok ? 1 : 0) != 0;
    };
    if (my > 0) prefetch(cta);
    for (int i = 0; i < my && !bad; ++i) {
        const int buf = a.nbuf == 2 ? (i & 1) : 0;
        if (a.nbuf == 1 && i > 0 && !wait_mma(i - 1)) {          // the single operand buffer is still being read
            bad = true;
            break;
        }
        store_stage(buf);
        fence_async_smem();
        fence_before_sync();
        __syncthreads();
        if (tid == 0) {
            fence_after_sync();
            issue(buf, i & 1);
        }
        if (i + 1 < my) prefetch(cta + (i + 1) * nctas);
        if (i > 0) {
            if (a.nbuf == 2 && !wait_mma(i - 1)) {
                bad = true;
                break;
            }
            fence_after_sync();
            epilogue(cta + (i - 1) * nctas, (i - 1) & 1);
        }
    }
    if (!bad && my > 0) {
        if (!wait_mma(my - 1)) bad = true;
        else {
            fence_after_sync();
            epilogue(cta + (my - 1) * nctas, (my - 1) & 1);
        }
    }
    if (bad && tid == 0) atomicExch(a.err, 1);
    fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 2 * C3P_NH);
}

// true if the persistent kernel takes the layer; fills its launch geometry
bool plan_c3p(const C3Args& a, C3PArgs& p, size_t* smem, int* it) {
    if (a.C > 128 || a.C % 64 || a.N % C3P_NH) return false;
    const int Wp = a.W + 2, rows = TM + 2 * Wp + 2;
    const int kbs = a.C / 64;
    *it = 8;                                            // items per thread: 256 threads x 8 chunks (C = 64) or 512 x 16 (C = 128)
    const int nthr = a.C == 64 ? 256 : 512;
    if (rows > *it * (nthr / (a.C >> 3))) return false;
    if ((double)a.n_img * a.H * a.W * (a.C > a.N ? a.C : a.N) / 8.0 >= 4.0e9) return false;      // 32-bit vector indices
    p.x = a.x; p.dz = a.dz; p.w = a.w; p.addend = a.addend; p.out = a.out; p.err = a.err;
    p.n_img = a.n_img; p.H = a.H; p.W = a.W; p.C = a.C; p.N = a.N; p.flip = a.flip;
    p.tiles_per_img = ((a.H - 1) * Wp + a.W + TM - 1) / TM;
    p.total_tiles = a.n_img * p.tiles_per_img;
    p.rows_pad = (rows + 7) / 8 * 8;
    p.n_split = a.N / C3P_NH;
    const size_t wbytes = 9 * (size_t)kbs * C3P_NH * 128, abuf = (size_t)kbs * p.rows_pad * 128;
    const size_t budget = 225 * 1024;
    p.nbuf = 1;
    *smem = wbytes + p.nbuf * abuf + 1024;
    return *smem <= (a.C == 64 ? budget / 2 : budget);
}

template <bool BWD> void launch_c3(C3Args& a, int kind, double bytes, double useful_flops, cudaStream_t st) {
    {
        C3PArgs p{};
        size_t psmem = 0;
        int it = 0;
        if (plan_c3p(a, p, &psmem, &it)) {
            smem_limit_once<106 + (BWD ? 50 : 0)>(conv3_persist_kernel<BWD, 8, 256>, 113 * 1024);
            smem_limit_once<107 + (BWD ? 50 : 0)>(conv3_persist_kernel<BWD, 8, 512>, 226 * 1024);
            const int n_sm = sm_count();
            const bool two = a.C == 64;                     // two 256-thread CTAs per SM
            int nctas = (two ? 2 * n_sm : n_sm) / p.n_split;
            if (nctas < 1) nctas = 1;
            if (nctas > p.total_tiles) nctas = p.total_tiles;
            LaunchScope ls(kind, bytes, useful_flops > 0 ? useful_flops : 2.0 * 9.0 * a.n_img * a.H * a.W * (double)a.C * a.N, st);
            if (two) launch_pdl(conv3_persist_kernel<BWD, 8, 256>, nctas * p.n_split, 256, psmem, st, p);
            else launch_pdl(conv3_persist_kernel<BWD, 8, 512>, nctas * p.n_split, 512, psmem, st, p);
            return;
        }
    }
    const int Wp = a.W + 2;
    const int centers = (a.H - 1) * Wp + a.W;           // positions Wp+1 .. H*Wp+W
    a.tiles_per_img = (centers + TM - 1) / TM;
    a.rows_pad = (TM + 2 * Wp + 2 + 7) / 8 * 8;
    a.tmem_cols = 32;
    while (a.tmem_cols < a.N) a.tmem_cols <<= 1;
    const int kbs = a.C / 64;
    // all nine taps resident if two CTAs per SM still fit with them
    a.resident = ((size_t)kbs * a.rows_pad * 128 + 9 * (size_t)kbs * a.N * 128 + 1024 <= 110 * 1024) ? 1 : 0;
    size_t smem = (size_t)kbs * a.rows_pad * 128 + (a.resident ? 9 : 2) * (size_t)kbs * a.N * 128 + 1024;
    smem_limit_once<108 + (BWD ? 50 : 0)>(conv3_tc_kernel<BWD>, 200 * 1024);
    LaunchScope ls(kind, bytes, useful_flops > 0 ? useful_flops : 2.0 * 9.0 * a.n_img * a.H * a.W * (double)a.C * a.N, st);
    launch_pdl(conv3_tc_kernel<BWD>, a.n_img * a.tiles_per_img, C3_THREADS, smem, st, a);
}


// ---------------------------------------------------------------------------------------------
// Weight gradient of the 3x3 conv:  gw[k][t][c] = sum_f dz[f][k] * x[f + off_t][c]  over the
// padded-flattened positions f of all images (dz and x are zero at padding positions).
// The reduction index is the position, so both operands are MN-major exactly as staged:
// rows = positions, 128 bytes = 64 channels.  x is staged with its halo once per tile and tap t
// reads it through a start address moved by off_t rows; each tap owns its own accumulator
// columns in tensor memory.  A CTA walks a range of tiles and a group of taps (9*c_in columns
// do not fit the 512 columns), accumulates in tensor memory, and writes one partial in the
// gradient's own layout; the partials are summed in index order by a second kernel.
struct W3Args {
    GradSrc dz;
    ValSrc x;
    float* partial;            // [ctas][CO][9][CI], only this CTA's taps are written
    int* err;
    int n_img, H, W, CI, CO;
    int tiles_per_img, total_tiles, tiles_per_cta, rows_pad, taps_per_group, tmem_cols;
};

__device__ __forceinline__ uint64_t make_desc_mn_lbo(uint32_t smem_addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

__global__ void __launch_bounds__(C3_THREADS) conv3_wgrad_tc_kernel(const W3Args a) {
    pdl_wait();
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_store;
    __shared__ uint32_t tmem_slot;
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Wp = a.W + 2;
    const int kbi = a.CI >> 6, kbo = (a.CO + 63) >> 6;
    const uint32_t x_block = (uint32_t)a.rows_pad * 128u;
    const uint32_t dz_block = TM * 128u;
    uint8_t* sDZ = base;                                   // two 64-channel panels (rows beyond c_out are never read back)
    uint8_t* sX = base + 2 * dz_block;
    const int rows = TM + 2 * Wp + 2;
    const uint32_t bar = smem_u32(&bar_store);
    const int t_first = blockIdx.y * a.taps_per_group;
    const int t_count = min(a.taps_per_group, 9 - t_first);
    if (tid == 0) mbar_init(bar, 1);
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), (uint32_t)a.tmem_cols);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    const uint32_t tmem = tmem_slot;
    const uint32_t idesc = make_idesc(a.CI) | (1u << 15) | (1u << 16);
    const int tile_beg = blockIdx.x * a.tiles_per_cta, tile_end = min(a.total_tiles, tile_beg + a.tiles_per_cta);
    uint32_t phase = 0;
    bool bad = false;
    const int vx = a.CI >> 3, vz = a.CO >> 3;             // chunks per row: 8 or 16, both divide 256
    const int jx = tid % vx, jz = tid % vz, stepx = C3_THREADS / vx, stepz = C3_THREADS / vz;
    const int sxq = stepx / Wp, sxr = stepx - sxq * Wp, szq = stepz / Wp, szr = stepz - szq * Wp;
    const bool need_z = a.dz.act != ACT_NONE || a.dz.k1 != nullptr;
    const uint4* gx = reinterpret_cast<const uint4*>(a.x.p);
    const uint4* gdy = reinterpret_cast<const uint4*>(a.dz.dy);
    const uint4* gz = reinterpret_cast<const uint4*>(a.dz.z);
    XfVal xv;
    XfGrad xg;
    xv.init(a.x, jx << 3);
    xg.init(a.dz, jz << 3);
    for (int tl = tile_beg; tl < tile_end; ++tl) {
        const int img = tl / a.tiles_per_img, tile = tl - img * a.tiles_per_img;
        const int f0 = Wp + 1 + tile * TM, fs0 = f0 - Wp - 1;
        // x with halo, then dz at the 128 centre positions: a thread owns one 16-byte channel chunk of each operand
        // (coefficients in registers) and every (256 / chunks)-th row; the loads of four rows are issued together
        {
            constexpr int U = 4;
            // (hp, wp) of consecutive items follow by additions (one division per tile and operand); 32-bit vector indices
            const uint32_t img_row0 = (uint32_t)img * (uint32_t)a.H;
            int hp = (fs0 + tid / vx) / Wp, wp = (fs0 + tid / vx) - hp * Wp;
            for (int rb = tid / vx; rb < rows; rb += U * stepx) {
                uint4 raw[U];
                bool ok[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = rb + u * stepx;
                    ok[u] = r < rows && (uint32_t)(hp - 1) < (uint32_t)a.H && (uint32_t)(wp - 1) < (uint32_t)a.W;
                    raw[u] = make_uint4(0, 0, 0, 0);
                    if (ok[u]) raw[u] = __ldg(gx + ((img_row0 + (uint32_t)(hp - 1)) * (uint32_t)a.W + (uint32_t)(wp - 1)) * (uint32_t)vx + (uint32_t)jx);
                    wp += sxr;
                    hp += sxq;
                    if (wp >= Wp) {
                        wp -= Wp;
                        ++hp;
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = rb + u * stepx;
                    if (r < rows) {
                        const uint4 q = ok[u] ? xv.apply(raw[u]) : make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4*>(sX + (size_t)(jx >> 3) * x_block + (size_t)r * 128 + ((((uint32_t)jx & 7u) ^ ((uint32_t)r & 7u)) << 4)) = q;
                    }
                }
            }
            hp = (f0 + tid / vz) / Wp;
            wp = (f0 + tid / vz) - hp * Wp;
            for (int rb = tid / vz; rb < TM; rb += U * stepz) {
                uint4 raw[U], rawz[U];
                bool ok[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = rb + u * stepz;
                    ok[u] = r < TM && (uint32_t)(hp - 1) < (uint32_t)a.H && (uint32_t)(wp - 1) < (uint32_t)a.W;
                    raw[u] = rawz[u] = make_uint4(0, 0, 0, 0);
                    if (ok[u]) {
                        const uint32_t e = ((img_row0 + (uint32_t)(hp - 1)) * (uint32_t)a.W + (uint32_t)(wp - 1)) * (uint32_t)vz + (uint32_t)jz;
                        raw[u] = __ldg(gdy + e);
                        if (need_z) rawz[u] = __ldg(gz + e);
                    }
                    wp += szr;
                    hp += szq;
                    if (wp >= Wp) {
                        wp -= Wp;
                        ++hp;
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int r = rb + u * stepz;
                    if (r < TM) {
                        uint4 q = make_uint4(0, 0, 0, 0);
                        if (ok[u]) q = need_z ? xg.apply(raw[u], rawz[u]) : raw[u];
                        *reinterpret_cast<uint4*>(sDZ + (size_t)(jz >> 3) * dz_block + (size_t)r * 128 + ((((uint32_t)jz & 7u) ^ ((uint32_t)r & 7u)) << 4)) = q;
                    }
                }
            }
        }
        fence_async_smem();
        __syncthreads();
        if (tid == 0) {
            fence_after_sync();
            const uint32_t z0 = smem_u32(sDZ), x0 = smem_u32(sX);
            for (int tt = 0; tt < t_count; ++tt) {
                const int t = t_first + tt, r = t / 3, s = t - r * 3;
                const uint32_t xs = x0 + (uint32_t)(r * Wp + s) * 128u;
                const uint32_t d = tmem + (uint32_t)(tt * a.CI);
                const uint64_t dz_const = make_desc_mn_lbo(0, dz_block), x_const = make_desc_mn_lbo(0, x_block);
#pragma unroll
                for (int k = 0; k < TM / 16; ++k)
                    umma_bf16(d, dz_const + (uint64_t)((z0 + k * 2048) >> 4), x_const + (uint64_t)((xs + k * 2048) >> 4), idesc,
                              (tl > tile_beg || k > 0) ? 1u : 0u);
            }
            umma_commit(bar);
        }
        bool ok = mbar_wait(bar, phase);      // shared memory is rewritten by the next tile
        phase ^= 1;
        if (!__syncthreads_and(ok ? 1 : 0)) {
            bad = true;
            break;
        }
    }
    fence_after_sync();
    __syncthreads();
    if (bad) {
        if (tid == 0) atomicExch(a.err, 1);
    } else {
        const int q = warp & 3, half = warp >> 2;
        const int k = q * 32 + lane;
        float* pb = a.partial + (size_t)blockIdx.x * a.CO * 9 * a.CI;
        for (int tt = 0; tt < t_count; ++tt) {
            const int t = t_first + tt;
            for (int g = half; g < (a.CI >> 4); g += 2) {
                float v[16];
                if (tile_end > tile_beg) {
                    tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(tt * a.CI + (g << 4)), v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
                if (k < a.CO) {
                    float* dst = pb + ((size_t)k * 9 + t) * a.CI + (g << 4);
#pragma unroll
                    for (int hh = 0; hh < 4; ++hh) *reinterpret_cast<float4*>(dst + hh * 4) = make_float4(v[hh * 4], v[hh * 4 + 1], v[hh * 4 + 2], v[hh * 4 + 3]);
                }
            }
        }
    }
    fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, (uint32_t)a.tmem_cols);
    (void)kbi; (void)kbo;
}

// out[i] = sum over splits of partial[split][i], n a multiple of 4.  A block finishes 128 consecutive outputs: warp kg adds
// the splits kg, kg+32, ... (each lane four consecutive outputs: 512 contiguous bytes per split and warp, all of a
// thread's loads issued before the additions), the 32 sub-sums are combined in index order through shared memory.
__global__ void __launch_bounds__(1024) reduce_splits_c3(const float* __restrict__ partial, int splits, size_t n, float* __restrict__ out) {
    pdl_wait();
    pdl_launch();
    __shared__ float4 sh[32][33];
    const int il = threadIdx.x & 31, kg = threadIdx.x >> 5;
    const size_t i = ((size_t)blockIdx.x * 32 + il) * 4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < n) {
        for (int k0 = kg; k0 < splits; k0 += 32 * 4) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                v[u] = (k0 + 32 * u < splits) ? *reinterpret_cast<const float4*>(partial + (size_t)(k0 + 32 * u) * n + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w;
            }
        }
    }
    sh[kg][il] = acc;
    __syncthreads();
    if (kg == 0 && i < n) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < 32; ++k) {
            const float4 v = sh[k][il];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        *reinterpret_cast<float4*>(out + i) = s;
    }
}

}  // namespace

void reduce_splits_f4(const float* partial, int splits, size_t n, float* out, cudaStream_t st) {
    launch_pdl(reduce_splits_c3, (unsigned)((n / 4 + 31) / 32), 1024, 0, st, partial, splits, n, out);
}

bool conv3_tc_supported(int dtype, const ConvGeom& g) {
    if (!(dtype == 1 && g.k == 3 && g.stride == 1 && g.pad == 1)) return false;
    if (g.ci % 64 || g.co % 64 || g.ci > 256 || g.co > 256) return false;
    const int Wp = g.wi + 2;
    const int rows_pad = (TM + 2 * Wp + 2 + 7) / 8 * 8;
    const int cmax = g.ci > g.co ? g.ci : g.co;
    return (size_t)(cmax / 64) * rows_pad * 128 + 2 * (size_t)(cmax / 64) * cmax * 128 + 1024 <= 200 * 1024;
}

void conv3_fwd_tc(const ConvGeom& g, const ValSrc& x, const __nv_bfloat16* wb, void* z, int* err, cudaStream_t st, double useful_flops) {
    C3Args a{};
    a.x = x; a.w = wb; a.out = (__nv_bfloat16*)z; a.err = err;
    a.n_img = g.n; a.H = g.hi; a.W = g.wi; a.C = g.ci; a.N = g.co; a.flip = 0;
    double px = (double)g.n * g.hi * g.wi;
    const double bytes = 2.0 * px * (g.ci + g.co) + 2.0 * 9 * g.ci * g.co;
    if (conv3_pipe(false, g.n, g.hi, g.wi, g.ci, g.co, x, GradSrc{}, wb, nullptr, z, err, K_CONV3_FWD_TC, bytes,
                   useful_flops > 0 ? useful_flops : 2.0 * 9.0 * px * g.ci * g.co, st))
        return;
    launch_c3<false>(a, K_CONV3_FWD_TC, bytes, useful_flops, st);
}

void conv3_bwd_data_tc(const ConvGeom& g, const GradSrc& dz, const __nv_bfloat16* wtb, const void* addend, void* dx, int* err, cudaStream_t st,
                       double useful_flops) {
    C3Args a{};
    a.dz = dz; a.w = wtb; a.addend = addend; a.out = (__nv_bfloat16*)dx; a.err = err;
    a.n_img = g.n; a.H = g.hi; a.W = g.wi; a.C = g.co; a.N = g.ci; a.flip = 1;
    double px = (double)g.n * g.hi * g.wi;
    const double bytes = 2.0 * px * g.co * ((dz.act != ACT_NONE || dz.k1) ? 2.0 : 1.0) + 2.0 * px * g.ci * (addend ? 2.0 : 1.0) + 2.0 * 9 * g.ci * g.co;
    if (conv3_pipe(true, g.n, g.hi, g.wi, g.co, g.ci, ValSrc{}, dz, wtb, addend, dx, err, K_CONV3_BWD_DATA_TC, bytes,
                   useful_flops > 0 ? useful_flops : 2.0 * 9.0 * px * g.ci * g.co, st))
        return;
    launch_c3<true>(a, K_CONV3_BWD_DATA_TC, bytes, useful_flops, st);
}

bool conv3_wgrad_tc_supported(int dtype, const ConvGeom& g) {
    // the kernel indexes 16-byte vectors with 32 bits
    return conv3_tc_supported(dtype, g) && g.ci <= 128 && g.co <= 128 && (double)g.n * g.hi * g.wi * 16.0 < 4.0e9;
}

void conv3_bwd_weight_tc(const ConvGeom& g, const GradSrc& dz, const ValSrc& x, float* scratch, size_t scratch_floats, float* gw, int* err,
                         cudaStream_t st, double useful_flops) {
    {
        // the pipelined kernel fed by tensor copies, where the layer fits it
        const double px = (double)g.n * g.hi * g.wi;
        const size_t out_elems = (size_t)g.co * 9 * g.ci;
        const int ctas = conv3_wgrad_pipe(g.n, g.hi, g.wi, g.ci, g.co, dz, x, scratch, scratch_floats, err,
                                          2.0 * px * g.co * ((dz.act != ACT_NONE || dz.k1) ? 2.0 : 1.0) + 2.0 * px * g.ci,
                                          useful_flops > 0 ? useful_flops : 2.0 * 9.0 * px * g.ci * g.co, st);
        if (ctas > 0) {
            LaunchScope ls(K_REDUCE_SPLITS, 4.0 * out_elems * (ctas + 1), (double)out_elems * ctas, st);
            launch_pdl(reduce_splits_c3, (unsigned)((out_elems / 4 + 31) / 32), 1024, 0, st, scratch, ctas, out_elems, gw);
            return;
        }
    }
    W3Args a{};
    a.dz = dz; a.x = x; a.partial = scratch; a.err = err;
    a.n_img = g.n; a.H = g.hi; a.W = g.wi; a.CI = g.ci; a.CO = g.co;
    const int Wp = a.W + 2;
    a.tiles_per_img = ((a.H - 1) * Wp + a.W + TM - 1) / TM;
    a.total_tiles = a.n_img * a.tiles_per_img;
    a.rows_pad = (TM + 2 * Wp + 2 + 7) / 8 * 8;
    // at most 256 accumulator columns per CTA, so that two CTAs of an SM hold their tensor memory at the same time and one
    // stages while the other multiplies: 3 taps x 64 channels (three groups) or 2 taps x 128 channels (five groups)
    a.taps_per_group = a.CI <= 64 ? 3 : 2;
    const int groups = (9 + a.taps_per_group - 1) / a.taps_per_group;
    a.tmem_cols = 32;
    while (a.tmem_cols < a.taps_per_group * a.CI) a.tmem_cols <<= 1;
    smem_limit_once<109>(conv3_wgrad_tc_kernel, 200 * 1024);
    const int n_sm = sm_count();
    const size_t out_elems = (size_t)a.CO * 9 * a.CI;
    int ctas = (2 * n_sm) / groups;
    if (ctas > a.total_tiles) ctas = a.total_tiles;
    if ((size_t)ctas > scratch_floats / out_elems) ctas = (int)(scratch_floats / out_elems);
    if (ctas < 1) ctas = 1;
    a.tiles_per_cta = (a.total_tiles + ctas - 1) / ctas;
    ctas = (a.total_tiles + a.tiles_per_cta - 1) / a.tiles_per_cta;
    size_t smem = 2 * (size_t)TM * 128 + (size_t)(a.CI / 64) * a.rows_pad * 128 + 1024;
    double px = (double)g.n * g.hi * g.wi;
    {
        LaunchScope ls(K_CONV3_BWD_WEIGHT_TC, 2.0 * px * g.co * ((dz.act != ACT_NONE || dz.k1) ? 2.0 : 1.0) + 2.0 * px * g.ci + 4.0 * out_elems,
                       useful_flops > 0 ? useful_flops : 2.0 * 9.0 * px * g.ci * g.co, st);
        launch_pdl(conv3_wgrad_tc_kernel, dim3(ctas, groups), C3_THREADS, smem, st, a);
    }
    LaunchScope ls(K_REDUCE_SPLITS, 4.0 * out_elems * (ctas + 1), (double)out_elems * ctas, st);
    launch_pdl(reduce_splits_c3, (unsigned)((out_elems / 4 + 31) / 32), 1024, 0, st, scratch, ctas, out_elems, gw);
}

}  // namespace ast
