// Dense 3x3 convolution (stride 1, pad 1), forward and backward-data, as a persistent
// warp-specialised implicit GEMM on tcgen05 fed by tiled bulk tensor copies.
//
// A tile is BH whole image rows.  Its operand is the (BH+2) x (W+2) window of input positions
// around it, one 64-channel block at a time, fetched by ONE 4-D tensor copy whose box starts at
// column -1 / row h0-1: positions outside the image arrive as zeros (the conv's padding), and the
// box lands in shared memory as consecutive 128-byte rows q = hh*(W+2) + wp in the swizzled
// K-major layout the MMA reads.  In these flattened padded coordinates tap (r,s) of output row
// m = oh*(W+2) + j reads operand row m + r*(W+2) + s: every tap is the same buffer seen through a
// descriptor moved by a constant number of rows, so a window is staged once for all nine taps.
// Output rows with j >= W are computed and dropped.
//
//   warp 0        producer: per (tile, channel block) one tensor copy of the raw window into a ring of slots (forward:
//                 the producing unit's raw output z; backward: dy, and z of the same window into a second ring)
//   warps 1-2     MMA issuers, alternating tiles, each into its own accumulator set in tensor memory: 9 taps x 4
//                 k-steps x MT row tiles of tcgen05.mma (N = 64) per window.  One issuing warp cannot keep the tensor
//                 pipe busy with instructions this small (the issue path, not the arithmetic, bounds a single warp);
//                 two reach the shared-memory bandwidth bound of an N = 64 instruction.  Every lane runs the loop
//                 (convergent control flow keeps the descriptor arithmetic in the uniform datapath), the elected
//                 lane issues.  The weights of the CTA's 64 output channels stay resident in shared memory for all
//                 taps (wider layers are split over CTAs by output channel).
//   warps 3-14    transform, IN PLACE on the landed window, all warps on the same window: BatchNorm + activation
//                 (forward) or the BatchNorm-backward transform of (dy, z) (backward) with per-thread register-held
//                 coefficients; padding positions are left as the zeros the copy wrote
//   warps 15-18   epilogue: tcgen05.ld, (+ residual gradient), round to bf16, 16-byte stores
//
// A parity wait on an mbarrier is only meaningful for a waiter that has seen the previous phase, so every warp of a
// role observes every window's phases in order and acknowledges them, whether or not it owns the window.
//
// Every wait is bounded; a wait that runs out raises a CTA-wide abort flag, all roles leave,
// copies in flight are waited for, tensor memory is freed and the error word is set.
#include <cuda_bf16.h>

#include "kernels.h"
#include "tc_common.cuh"
#include "tma.cuh"

namespace ast {
namespace {

using namespace tc;
constexpr int CP_XF_WARPS = 12, CP_EPI_WARPS = 4;
constexpr int CP_MMA_WARPS = 2;
constexpr int CP_FIRST_XF = 1 + CP_MMA_WARPS;
constexpr int CP_THREADS = (CP_FIRST_XF + CP_XF_WARPS + CP_EPI_WARPS) * 32;
constexpr int CP_NH = 64;              // output channels per CTA
constexpr int CP_NI = 5;               // window rows a transform thread owns at most: (BH+2)*(W+2) <= 48 * CP_NI
constexpr int CP_MAX_S = 4;            // operand ring slots
constexpr uint32_t CP_WTAP = CP_NH * 128u;   // bytes of one tap's weights for one 64-channel block

struct CPArgs {
    ValSrc x;                  // forward: coefficient pointers and activation (data come through the tensor map)
    GradSrc dz;                // backward: likewise
    const void* addend;        // backward only, may be null: [n][H][W][N]
    __nv_bfloat16* out;        // [n][H][W][N]
    int* err;
    int n_img, H, W, C, N;     // C: reduction channels (64 or 128), N: output channels (multiple of 64)
    int BH, MT;                // image rows per tile; 128-row MMA tiles per tile (1 or 2)
    int tiles_per_img, total_tiles, n_split, flip;
    int S, ZS;                 // ring depths: operand windows; z windows (backward with a transform)
    uint32_t zslot_bytes;      // bytes of one z ring slot (multiple of 1024)
    uint32_t slot_bytes;       // bytes of one ring slot (multiple of 1024)
    uint32_t box_bytes;        // bytes one tensor copy delivers: 128 * (W+2) * (BH+2)
    int need_xf;               // the window needs a transform
};

template <bool BWD>
__global__ void __launch_bounds__(CP_THREADS, 1)
conv3_pipe_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_z, const __grid_constant__ CUtensorMap tm_w,
                  const CPArgs a) {
    // barriers, tensor memory and the resident weights (written only by the refresh kernel, which never releases its
    // dependents early) are set up before the dependency wait and overlap the previous kernel's tail
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    // w_full, slot_full[S], slot_xf[S], slot_empty[S], acc_full[2], acc_empty[2], z_full[2], z_empty[2]
    __shared__ uint64_t bars[1 + 3 * CP_MAX_S + 8];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_store;
    volatile int* abort_flag = &abort_store;
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Wp = a.W + 2, kbs = a.C >> 6, S = a.S, MT = a.MT;
    const uint32_t wbytes = (uint32_t)kbs * 9u * CP_WTAP;
    uint8_t* sB = base;
    uint8_t* sA = sB + wbytes;
    uint8_t* sZ = sA + (size_t)S * a.slot_bytes;
    const int ZS = a.ZS;
    const bool use_z = BWD && a.need_xf;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto w_full = [&]() { return bar0; };
    auto slot_full = [&](int s) { return bar0 + 8u * (1 + s); };
    auto slot_xf = [&](int s) { return bar0 + 8u * (1 + CP_MAX_S + s); };
    auto slot_empty = [&](int s) { return bar0 + 8u * (1 + 2 * CP_MAX_S + s); };
    auto acc_full = [&](int s) { return bar0 + 8u * (1 + 3 * CP_MAX_S + s); };
    auto acc_empty = [&](int s) { return bar0 + 8u * (1 + 3 * CP_MAX_S + 2 + s); };
    auto z_full = [&](int s) { return bar0 + 8u * (1 + 3 * CP_MAX_S + 4 + s); };
    auto z_empty = [&](int s) { return bar0 + 8u * (1 + 3 * CP_MAX_S + 6 + s); };
    const int half = blockIdx.x % a.n_split, n0 = half * CP_NH;
    const int cta = blockIdx.x / a.n_split, nctas = gridDim.x / a.n_split;
    const int my_tiles = cta < a.total_tiles ? (a.total_tiles - cta + nctas - 1) / nctas : 0;
    const int total_items = my_tiles * kbs;
    const uint32_t tmem_cols = MT == 2 ? 256u : 128u;

    if (tid == 0) {
        mbar_init(w_full(), 1);
        for (int s = 0; s < CP_MAX_S; ++s) {
            mbar_init(slot_full(s), 1);
            mbar_init(slot_xf(s), CP_XF_WARPS);
            mbar_init(slot_empty(s), CP_MMA_WARPS);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(z_full(s), 1);
            mbar_init(z_empty(s), CP_XF_WARPS);
            mbar_init(acc_full(s), 1);
            mbar_init(acc_empty(s), CP_EPI_WARPS);
        }
        abort_store = 0;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    if (tid == 0) {
        tma::prefetch_map(&tm_w);
        tma::prefetch_map(&tm_a);
        mbar_expect_tx(w_full(), wbytes);
        for (int kb = 0; kb < kbs; ++kb)
            for (int t = 0; t < 9; ++t)
                tma::load_3d(smem_u32(sB) + (uint32_t)(kb * 9 + t) * CP_WTAP, &tm_w, kb * 64, (a.flip) ? 8 - t : t, n0, w_full());
    }
    pdl_wait();
    const uint32_t tmem = tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            int it = 0, zit = 0;             // operand / z window copies issued
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tl = cta + t * nctas;
                const int img = tl / a.tiles_per_img, h0 = (tl - img * a.tiles_per_img) * a.BH;
                for (int kb = 0; kb < kbs; ++kb) {
                    const int s = it % S, n = it / S;
                    if (n > 0 && !mbar_wait_abortable(slot_empty(s), (uint32_t)((n - 1) & 1), abort_flag)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(slot_full(s), a.box_bytes);
                    tma::load_4d(smem_u32(sA + (size_t)s * a.slot_bytes), &tm_a, kb * 64, -1, h0 - 1, img, slot_full(s));
                    if (use_z) {
                        const int zs = it % ZS, zn = it / ZS;
                        if (zn > 0 && !mbar_wait_abortable(z_empty(zs), (uint32_t)((zn - 1) & 1), abort_flag)) {
                            ++it;      // the operand copy of this window is in flight: the drain below waits for it
                            ok = false;
                            break;
                        }
                        mbar_expect_tx(z_full(zs), a.box_bytes);
                        tma::load_4d(smem_u32(sZ + (size_t)zs * a.zslot_bytes), &tm_z, kb * 64, -1, h0 - 1, img, z_full(zs));
                        ++zit;
                    }
                    ++it;
                }
            }
            // never leave while a copy into this CTA's shared memory may still be in flight
            for (int k = (it > S ? it - S : 0); k < it; ++k) mbar_wait(slot_full(k % S), (uint32_t)((k / S) & 1));
            for (int k = (zit > ZS ? zit - ZS : 0); k < zit; ++k) mbar_wait(z_full(k % ZS), (uint32_t)((k / ZS) & 1));
            mbar_wait(w_full(), 0);
        }
    } else if (warp < CP_FIRST_XF) {
        // ------------------------------------------------------------ MMA issuers: warp w takes tiles w-1, w+1, ... into accumulator set w-1
        {
            const int iss = warp - 1;
            const uint32_t leader = elect_leader();
            const uint32_t idesc = make_idesc(CP_NH);
            const uint64_t dconst = make_desc(0);
            const uint32_t b0 = smem_u32(sB) >> 4;
            bool ok = mbar_wait_abortable(w_full(), 0, abort_flag);
            // Both issuer warps observe every window's barrier phase in order and acknowledge it (a parity wait is only
            // meaningful for a waiter that has seen the previous phase); the owner of the window's tile issues its MMAs.
            for (int it = 0; it < total_items && ok; ++it) {
                const int t = it / kbs, kb = it - t * kbs;
                const bool mine = (t % CP_MMA_WARPS) == iss;
                const int s = it % S, b = t & 1, n = t >> 1;
                if (mine && kb == 0 && n > 0 && !mbar_wait_abortable(acc_empty(b), (uint32_t)((n - 1) & 1), abort_flag)) break;
                if (!mbar_wait_abortable(slot_xf(s), (uint32_t)((it / S) & 1), abort_flag)) break;
                if (mine) {
                    fence_after_sync();
                    const uint32_t a0 = smem_u32(sA + (size_t)s * a.slot_bytes) >> 4;
                    for (int mt = 0; mt < MT; ++mt) {
                        const uint32_t d = tmem + (uint32_t)((b * MT + mt) * CP_NH);
#pragma unroll
                        for (int tp = 0; tp < 9; ++tp) {
                            const int r = tp / 3, sx = tp - r * 3;
                            const uint32_t ar = a0 + (uint32_t)(mt * TM + r * Wp + sx) * 8u;      // 128-byte rows, in 16-byte units
                            const uint32_t br = b0 + (uint32_t)(kb * 9 + tp) * (CP_WTAP >> 4);
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                umma_bf16_lead(d, dconst + (uint64_t)(ar + 2u * ks), dconst + (uint64_t)(br + 2u * ks), idesc, (kb > 0 || tp > 0 || ks > 0) ? 1u : 0u, leader);
                        }
                    }
                    umma_commit_lead(slot_empty(s), leader);
                    if (kb == kbs - 1) umma_commit_lead(acc_full(b), leader);
                } else if (leader) {
                    mbar_arrive(slot_empty(s));
                }
                __syncwarp();
            }
        }
    } else if (warp < CP_FIRST_XF + CP_XF_WARPS) {
        // ------------------------------------------------------------ transform (in place)
        // All transform warps work on the same window: thread (pos0, j) owns 16-byte chunk j of window rows pos0,
        // pos0 + 48, ... (at most CP_NI of them).  Row geometry does not depend on the window and is computed once.
        // Backward: dy sits in the slot, z in the matching z ring slot (same row layout).
        const int xt = tid - CP_FIRST_XF * 32;
        const int j = xt & 7, pos0 = xt >> 3;
        constexpr int NPOS = CP_XF_WARPS * 4;                // window rows per pass
        const int rows = (a.BH + 2) * Wp;
        // 48 rows are a multiple of 8: the swizzle term of a thread's chunk is the same in all its rows
        const uint32_t off0 = (uint32_t)pos0 * 128u + (uint32_t)((j ^ (pos0 & 7)) << 4);
        int hw[CP_NI];                                       // (image row of the window << 16) | image column, or -1: padding column / beyond the window
#pragma unroll
        for (int i = 0; i < CP_NI; ++i) {
            const int q = pos0 + NPOS * i;
            const int hh = q / Wp, wp = q - hh * Wp;
            hw[i] = (q < rows && wp >= 1 && wp <= a.W) ? ((hh << 16) | (wp - 1)) : -1;
        }
        XfVal xv;
        XfGrad xg;
        if (a.need_xf && kbs == 1) {
            if (BWD) xg.init(a.dz, j << 3);
            else xv.init(a.x, j << 3);
        }
        for (int it = 0; it < total_items; ++it) {
            const int s = it % S;
            const int t = it / kbs, kb = it - t * kbs;
            const int tl = cta + t * nctas;
            const int img = tl / a.tiles_per_img, h0 = (tl - img * a.tiles_per_img) * a.BH;
            if (a.need_xf && kbs > 1) {                      // the channel block changes from window to window
                if (BWD) xg.init(a.dz, kb * 64 + (j << 3));
                else xv.init(a.x, kb * 64 + (j << 3));
            }
            if (!mbar_wait_abortable(slot_full(s), (uint32_t)((it / S) & 1), abort_flag)) break;
            const int zs = it % ZS;
            if (use_z && !mbar_wait_abortable(z_full(zs), (uint32_t)((it / ZS) & 1), abort_flag)) break;
            if (a.need_xf) {
                uint8_t* slot = sA + (size_t)s * a.slot_bytes + off0;
                const uint8_t* zslot = sZ + (size_t)zs * a.zslot_bytes + off0;
#pragma unroll
                for (int i = 0; i < CP_NI; ++i) {
                    if (hw[i] >= 0 && (uint32_t)(h0 - 1 + (hw[i] >> 16)) < (uint32_t)a.H) {
                        uint4* p = reinterpret_cast<uint4*>(slot + (uint32_t)(NPOS * 128 * i));
                        *p = BWD ? xg.apply(*p, *reinterpret_cast<const uint4*>(zslot + (uint32_t)(NPOS * 128 * i))) : xv.apply(*p);
                    }
                }
                fence_async_smem();
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(slot_xf(s));
                if (use_z) mbar_arrive(z_empty(zs));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;                              // tensor-memory lane quarter of this warp
        for (int t = 0; t < my_tiles; ++t) {
            const int b = t & 1, n = t >> 1;
            const int tl = cta + t * nctas;
            const int img = tl / a.tiles_per_img, h0 = (tl - img * a.tiles_per_img) * a.BH;
            if (!mbar_wait_abortable(acc_full(b), (uint32_t)(n & 1), abort_flag)) break;
            fence_after_sync();
            for (int mt = 0; mt < MT; ++mt) {
                const int m = mt * TM + q * 32 + lane;
                const int oh = m / Wp, jj = m - oh * Wp;
                const bool pix = oh < a.BH && jj < a.W && h0 + oh < a.H;
                uint32_t rr[4][16];
#pragma unroll
                for (int u = 0; u < 4; ++u) tmem_ld16_issue(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)((b * MT + mt) * CP_NH + (u << 4)), rr[u]);
                tmem_ld_wait();
#pragma unroll
                for (int u = 0; u < 4; ++u) tmem_ld_pin16(rr[u]);
                if (pix) {
                    const size_t e0 = (((size_t)img * a.H + (h0 + oh)) * a.W + jj) * a.N + n0;
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            float vv[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) vv[i] = __uint_as_float(rr[u][(hh << 3) + i]);
                            const size_t e = e0 + (u << 4) + (hh << 3);
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
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(b));
        }
    }
    fence_before_sync();
    __syncthreads();
    if (tid == 0 && abort_store) atomicExch(a.err, 1);
    if (warp == 1) tmem_dealloc(tmem, tmem_cols);
}

// Geometry of the pipelined kernel for one layer; false if the layer does not fit it.
bool plan_cp(bool zring, int n_img, int H, int W, int C, int N, CPArgs& p, size_t* smem) {
    if (C % 64 || C > 128 || N % CP_NH || W + 2 > 126 || H < 1) return false;
    const int Wp = W + 2, kbs = C / 64;
    const size_t wbytes = (size_t)kbs * 9 * CP_WTAP;
    const size_t budget = 226 * 1024 - 1024;
    const int n_split = N / CP_NH;
    const int nctas = sm_count() / n_split > 0 ? sm_count() / n_split : 1;
    double best = 0;
    bool found = false;
    for (int bh = 1; bh <= H && bh * Wp <= 2 * TM && bh + 2 <= 256; ++bh) {
        const int mt = (bh * Wp + TM - 1) / TM;
        int rows = (bh + 2) * Wp;                       // the window the copy delivers
        if (rows < mt * TM + 2 * Wp + 2) rows = mt * TM + 2 * Wp + 2;      // the rows the last tap of the last MMA row reads
        rows = (rows + 7) / 8 * 8;
        const size_t slot = (size_t)rows * 128;
        if ((bh + 2) * Wp > CP_XF_WARPS * 4 * CP_NI) continue;      // the transform threads' share of a window
        // backward with a transform: z windows (only the rows the copy delivers) in a ring of their own
        const size_t zslot = zring ? ((size_t)(bh + 2) * Wp * 128 + 1023) / 1024 * 1024 : 0;
        if (wbytes + 2 * slot + zslot > budget) continue;
        int zs = zring ? 1 : 0;
        if (zring && wbytes + 2 * slot + 2 * zslot <= budget) zs = 2;
        int s = (int)((budget - wbytes - zs * zslot) / slot);
        if (s > CP_MAX_S) s = CP_MAX_S;
        const int tiles = n_img * ((H + bh - 1) / bh);
        const int iters = (tiles + nctas - 1) / nctas;
        // time model: MMA time per window (MT row tiles) plus a fixed hand-off cost; a deeper ring hides more latency
        const double cost = iters * (mt * 1.0 + 0.25) * (s >= 3 ? 1.0 : 1.15) * (zring && zs < 2 ? 1.2 : 1.0);
        if (!found || cost < best) {
            found = true;
            best = cost;
            p.BH = bh;
            p.MT = mt;
            p.S = s;
            p.ZS = zs > 0 ? zs : 1;
            p.zslot_bytes = (uint32_t)zslot;
            p.slot_bytes = (uint32_t)slot;
            p.box_bytes = 128u * (uint32_t)Wp * (uint32_t)(bh + 2);
            p.tiles_per_img = (H + bh - 1) / bh;
            p.total_tiles = tiles;
            *smem = wbytes + (size_t)s * slot + zs * zslot + 1024;
        }
    }
    p.n_split = n_split;
    return found;
}

bool make_maps(const void* act, const void* zt, const void* w, int n_img, int H, int W, int C, int N, int BH, CUtensorMap* ma, CUtensorMap* mz, CUtensorMap* mw) {
    const uint64_t dims[4] = {(uint64_t)C, (uint64_t)W, (uint64_t)H, (uint64_t)n_img};
    const uint64_t strides[3] = {(uint64_t)C * 2, (uint64_t)W * C * 2, (uint64_t)H * W * C * 2};
    const uint32_t box[4] = {64, (uint32_t)(W + 2), (uint32_t)(BH + 2), 1};
    if (!tma::encode_bf16(ma, act, 4, dims, strides, box)) return false;
    if (!tma::encode_bf16(mz, zt ? zt : act, 4, dims, strides, box)) return false;
    // weights [N][9][C]: dims {C, 9, N}; one copy = one tap of 64 output channels and 64 reduction channels
    const uint64_t wd[3] = {(uint64_t)C, 9, (uint64_t)N};
    const uint64_t ws[2] = {(uint64_t)C * 2, (uint64_t)9 * C * 2};
    const uint32_t wb[3] = {64, 1, CP_NH};
    return tma::encode_bf16(mw, w, 3, wd, ws, wb);
}

}  // namespace

// Forward (bwd == false: src = x, w = [c_out][9][c_in]) or backward-data (bwd == true: g = dz, w = [c_in][9][c_out],
// taps flipped) of a stride-1 3x3 conv through the pipelined kernel.  Returns false (nothing launched) if the layer does not fit.
bool conv3_pipe(bool bwd, int n_img, int H, int W, int C, int N, const ValSrc& x, const GradSrc& dz, const __nv_bfloat16* w, const void* addend,
                void* out, int* err, int kind, double bytes, double flops, cudaStream_t st) {
    CPArgs p{};
    size_t smem = 0;
    if ((double)n_img * H * W * (double)(C > N ? C : N) >= 2.0e9) return false;
    const bool need_xf = bwd ? grad_needs_z(dz) : (x.scale != nullptr || x.act != ACT_NONE);
    if (!plan_cp(bwd && need_xf, n_img, H, W, C, N, p, &smem)) return false;
    p.x = x; p.dz = dz; p.addend = addend; p.out = (__nv_bfloat16*)out; p.err = err;
    p.n_img = n_img; p.H = H; p.W = W; p.C = C; p.N = N; p.flip = bwd ? 1 : 0;
    p.need_xf = need_xf ? 1 : 0;
    alignas(64) CUtensorMap ma, mz, mw;
    if (!make_maps(bwd ? dz.dy : x.p, bwd && need_xf ? dz.z : nullptr, w, n_img, H, W, C, N, p.BH, &ma, &mz, &mw)) return false;
    smem_limit_once<120>(conv3_pipe_kernel<false>, 226 * 1024);
    smem_limit_once<121>(conv3_pipe_kernel<true>, 226 * 1024);
    int nctas = sm_count() / p.n_split;
    if (nctas < 1) nctas = 1;
    if (nctas > p.total_tiles) nctas = p.total_tiles;
    LaunchScope ls(kind, bytes, flops, st);
    if (bwd) launch_pdl(conv3_pipe_kernel<true>, nctas * p.n_split, CP_THREADS, smem, st, ma, mz, mw, p);
    else launch_pdl(conv3_pipe_kernel<false>, nctas * p.n_split, CP_THREADS, smem, st, ma, mz, mw, p);
    return true;
}

}  // namespace ast
