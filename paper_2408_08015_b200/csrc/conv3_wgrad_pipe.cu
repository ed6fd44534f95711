// Weight gradient of the dense 3x3 convolution (stride 1, pad 1) as a persistent warp-specialised
// pipeline on tcgen05 fed by tiled bulk tensor copies.
//
//   gw[k][t][c] = sum_m dz[m][k] * x[m + off_t][c],   off_t = r*(W+2) + s
//
// over the padded, flattened positions m = oh*(W+2) + j of a tile of BH image rows (dz is zero at
// the two junk columns j >= W of every row).  The reduction index is the position, so both
// operands are read exactly as the tensor copies deliver them, rows = positions of 128 bytes =
// 64 channels (MN-major for the MMA): the x window of (BH+2) x (W+2) positions arrives with its
// zero padding from a box that starts at column -1 / row h0-1, the dy and z windows of BH x (W+2)
// positions from boxes that start at column 0 and run two columns past the image (zeros).  Tap t
// reads the x window through a descriptor moved by off_t rows.  Every tap owns c_in accumulator
// columns in tensor memory; nine taps do not fit the 512 columns, so the taps are split over
// groups of CTAs (each group stages the same windows), and a CTA accumulates over all its tiles
// and writes one partial in the gradient's own layout; the partials are summed in index order by
// the split-sum kernel.
//
//   warp 0        producer: per tile the tensor copies of x and dy (one ring) and of z (a second ring)
//   warps 1-2     MMA issuers: each owns a share of the CTA's taps (disjoint accumulator columns) and
//                 issues, for every 16 positions, one tcgen05.mma (M = 128 output channels, N = c_in)
//                 per tap; every lane runs the loop, the elected lane issues
//   warps 3-6     transform x in place (BatchNorm + activation), padding positions stay zero
//   warps 7-14    transform dy in place into dz (BatchNorm-backward transform with z); where only one operand needs a
//                 transform all twelve warps work on it
//   warps 15-18   after the last tile: tcgen05.ld of the accumulators, float stores of the partial
//
// Shared memory is zeroed once: rows of a slot that no copy ever writes (the tail up to a whole
// number of 16-position steps, the rows the last taps read past the window) are multiplied by
// zeros of the other operand and must be finite.  Every wait is bounded and reports through the
// error word.
#include <cuda_bf16.h>

#include "kernels.h"
#include "tc_common.cuh"
#include "tma.cuh"

namespace ast {
namespace {

using namespace tc;
// 19 warps: with more, the register allocation per thread drops below what the backward transform's coefficients need and
// they spill into the hot loop
constexpr int WP_X_WARPS = 4, WP_D_WARPS = 8, WP_EPI_WARPS = 4, WP_MMA_WARPS = 2;
constexpr int WP_FIRST_X = 1 + WP_MMA_WARPS, WP_FIRST_D = WP_FIRST_X + WP_X_WARPS, WP_FIRST_EPI = WP_FIRST_D + WP_D_WARPS;
constexpr int WP_THREADS = (WP_FIRST_EPI + WP_EPI_WARPS) * 32;
constexpr int WP_MAX_S = 3;

struct WPArgs {
    ValSrc x;
    GradSrc dz;
    float* partial;            // [ctas per group][CO][9][CI]; a CTA writes its group's taps
    int* err;
    int n_img, H, W, CI, CO;
    int BH, ksteps;            // image rows per tile; 16-position steps per tile
    int tiles_per_img, total_tiles;
    int taps_per_group;        // taps per CTA group (blockIdx.y)
    int S, ZS;                 // ring depths: (x, dy) stages and z stages
    uint32_t x_block, d_block; // bytes of one 64-channel block of the x window / of the dy (z) window, multiples of 1024
    uint32_t stage_bytes;      // (CI/64) * x_block + (CO/64) * d_block
    uint32_t z_bytes;          // (CO/64) * d_block
    uint32_t x_box, d_box;     // bytes one copy delivers
    uint32_t smem_bytes;       // all ring memory (zeroed at start)
    uint32_t tmem_cols;
    int xf_x, xf_d;            // the operands need a transform
};

__device__ __forceinline__ uint64_t desc_mn(uint32_t smem_addr, uint32_t lbo_bytes) {
    // MN-major, 128-byte swizzle: leading-dimension offset = distance between 64-channel panels, stride-dimension offset =
    // 1024 bytes between groups of 8 positions
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

__global__ void __launch_bounds__(WP_THREADS, 1)
conv3_wgrad_pipe_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_dy, const __grid_constant__ CUtensorMap tm_z,
                        const WPArgs a) {
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    // st_full[S], st_xf[S], st_empty[S], z_full[2], z_empty[2], done
    __shared__ uint64_t bars[3 * WP_MAX_S + 5];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_store;
    volatile int* abort_flag = &abort_store;
    // 1024-byte aligned start, formed by pointer arithmetic on the shared array: a round trip through an integer would make
    // every access through it a generic load / store instead of a shared-memory one
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Wp = a.W + 2, kbi = a.CI >> 6, kbo = a.CO >> 6, S = a.S, ZS = a.ZS;
    uint8_t* sSt = base;                                   // stages: [x blocks][dy blocks]
    uint8_t* sZ = base + (size_t)S * a.stage_bytes;        // z stages
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto st_full = [&](int s) { return bar0 + 8u * s; };
    auto st_xf = [&](int s) { return bar0 + 8u * (WP_MAX_S + s); };
    auto st_empty = [&](int s) { return bar0 + 8u * (2 * WP_MAX_S + s); };
    auto z_full = [&](int s) { return bar0 + 8u * (3 * WP_MAX_S + s); };
    auto z_empty = [&](int s) { return bar0 + 8u * (3 * WP_MAX_S + 2 + s); };
    const uint32_t done = bar0 + 8u * (3 * WP_MAX_S + 4);
    const int cta = blockIdx.x, nctas = gridDim.x;
    const int t_first = blockIdx.y * a.taps_per_group;
    const int t_count = min(a.taps_per_group, 9 - t_first);
    const int my_tiles = cta < a.total_tiles ? (a.total_tiles - cta + nctas - 1) / nctas : 0;
    const bool use_z = a.xf_d != 0;

    if (tid == 0) {
        for (int s = 0; s < WP_MAX_S; ++s) {
            mbar_init(st_full(s), 1);
            mbar_init(st_xf(s), WP_X_WARPS + WP_D_WARPS);
            mbar_init(st_empty(s), WP_MMA_WARPS);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(z_full(s), 1);
            mbar_init(z_empty(s), a.xf_x ? WP_D_WARPS : WP_X_WARPS + WP_D_WARPS);
        }
        mbar_init(done, WP_MMA_WARPS);
        abort_store = 0;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_slot), a.tmem_cols);
        tmem_relinquish();
    }
    // rows no copy writes must hold finite values (they meet zeros of the other operand): zero everything once
    for (uint32_t o = (uint32_t)tid * 16u; o < a.smem_bytes; o += WP_THREADS * 16u) *reinterpret_cast<uint4*>(base + o) = make_uint4(0, 0, 0, 0);
    fence_async_smem();
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
    if (tid == 0) {
        tma::prefetch_map(&tm_x);
        tma::prefetch_map(&tm_dy);
        if (use_z) tma::prefetch_map(&tm_z);
    }
    pdl_wait();
    const uint32_t tmem = tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            int it = 0, zit = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int tl = cta + t * nctas;
                const int img = tl / a.tiles_per_img, h0 = (tl - img * a.tiles_per_img) * a.BH;
                const int s = it % S, n = it / S;
                if (n > 0 && !mbar_wait_abortable(st_empty(s), (uint32_t)((n - 1) & 1), abort_flag)) break;
                uint8_t* st = sSt + (size_t)s * a.stage_bytes;
                mbar_expect_tx(st_full(s), (uint32_t)kbi * a.x_box + (uint32_t)kbo * a.d_box);
                for (int kb = 0; kb < kbi; ++kb) tma::load_4d(smem_u32(st + (size_t)kb * a.x_block), &tm_x, kb * 64, -1, h0 - 1, img, st_full(s));
                for (int kb = 0; kb < kbo; ++kb)
                    tma::load_4d(smem_u32(st + (size_t)kbi * a.x_block + (size_t)kb * a.d_block), &tm_dy, kb * 64, 0, h0, img, st_full(s));
                ++it;
                if (use_z) {
                    const int zs = zit % ZS, zn = zit / ZS;
                    if (zn > 0 && !mbar_wait_abortable(z_empty(zs), (uint32_t)((zn - 1) & 1), abort_flag)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(z_full(zs), (uint32_t)kbo * a.d_box);
                    for (int kb = 0; kb < kbo; ++kb) tma::load_4d(smem_u32(sZ + (size_t)zs * a.z_bytes + (size_t)kb * a.d_block), &tm_z, kb * 64, 0, h0, img, z_full(zs));
                    ++zit;
                }
            }
            // never leave while a copy into this CTA's shared memory may still be in flight
            for (int k = (it > S ? it - S : 0); k < it; ++k) mbar_wait(st_full(k % S), (uint32_t)((k / S) & 1));
            for (int k = (zit > ZS ? zit - ZS : 0); k < zit; ++k) mbar_wait(z_full(k % ZS), (uint32_t)((k / ZS) & 1));
        }
    } else if (warp < WP_FIRST_X) {
        // ------------------------------------------------------------ MMA issuers
        const int iss = warp - 1;
        const uint32_t leader = elect_leader();
        // D = f32, A = B = bf16, both MN-major (bits 15, 16); M = 128, N = c_in
        const uint32_t idesc = make_idesc(a.CI) | (1u << 15) | (1u << 16);
        const uint32_t idesc2 = make_idesc(2 * a.CI) | (1u << 15) | (1u << 16);      // a pair of taps (64 input channels)
        // this warp's taps of the group: the first ceil(n/2) or the rest
        const int h = (t_count + 1) >> 1;
        const int tt0 = iss == 0 ? 0 : h, tt1 = iss == 0 ? h : t_count;
        // with 64 output channels the second 64-row panel of the A operand repeats the first (leading-dimension offset 0);
        // its accumulator rows are never read
        const uint32_t lbo_a = kbo > 1 ? a.d_block : 0u, lbo_b = kbi > 1 ? a.x_block : 128u;
        bool ok = true;
        for (int t = 0; t < my_tiles && ok; ++t) {
            const int s = t % S;
            if (!mbar_wait_abortable(st_xf(s), (uint32_t)((t / S) & 1), abort_flag)) {
                ok = false;
                break;
            }
            fence_after_sync();
            const uint32_t x0 = smem_u32(sSt + (size_t)s * a.stage_bytes);
            const uint32_t d0 = x0 + (uint32_t)kbi * a.x_block;
            for (int tt = tt0; tt < tt1;) {
                const int tp = t_first + tt, r = tp / 3, sx = tp - r * 3;
                const uint32_t xs = x0 + (uint32_t)(r * Wp + sx) * 128u;
                const uint32_t d = tmem + (uint32_t)(tt * a.CI);
                if (kbi == 1 && tt + 1 < tt1) {
                    // 64 input channels: two consecutive taps in one instruction of N = 128.  The second 64-column panel of the B
                    // operand is the same x window moved by the distance between the two taps' row offsets (the
                    // leading-dimension offset), its accumulator columns are the next tap's: half the instructions, and the A
                    // operand is fetched from shared memory once for both taps.
                    const uint32_t lbo_pair = (uint32_t)(sx < 2 ? 1 : Wp - 2) * 128u;
                    for (int k = 0; k < a.ksteps; ++k)
                        umma_bf16_lead(d, desc_mn(d0 + (uint32_t)k * 2048u, lbo_a), desc_mn(xs + (uint32_t)k * 2048u, lbo_pair), idesc2, (t > 0 || k > 0) ? 1u : 0u,
                                       leader);
                    tt += 2;
                } else {
                    for (int k = 0; k < a.ksteps; ++k)
                        umma_bf16_lead(d, desc_mn(d0 + (uint32_t)k * 2048u, lbo_a), desc_mn(xs + (uint32_t)k * 2048u, lbo_b), idesc, (t > 0 || k > 0) ? 1u : 0u, leader);
                    tt += 1;
                }
            }
            umma_commit_lead(st_empty(s), leader);
            __syncwarp();
        }
        if (ok) umma_commit_lead(done, leader);
    } else if (warp < WP_FIRST_EPI) {
        // ------------------------------------------------------------ transforms, in place
        // Split of the twelve transform warps: four on x and eight on dy when both operands need a transform, all twelve on
        // the one that does when only one does (a stride-2 layer's zero-inserted gradient arrives already transformed)
        const int wt = warp - WP_FIRST_X;
        const bool both = a.xf_x && a.xf_d;
        const bool is_x = both ? wt < WP_X_WARPS : a.xf_x != 0;
        const int nrole = both ? (is_x ? WP_X_WARPS : WP_D_WARPS) : WP_X_WARPS + WP_D_WARPS;
        const int nblk = is_x ? kbi : kbo;                       // channel blocks of this operand
        const int nw = nrole / nblk;                             // warps per block
        const int wi = both && !is_x ? wt - WP_X_WARPS : wt;
        const int kb = wi / nw, wl = wi - kb * nw;               // this warp's block; its index among the block's warps
        const int j = lane & 7, pos0 = wl * 4 + (lane >> 3), npos = nw * 4;
        const bool need = is_x ? a.xf_x != 0 : a.xf_d != 0;
        XfVal xv;
        XfGrad xg;
        if (need) {
            if (is_x) xv.init(a.x, kb * 64 + (j << 3));
            else xg.init(a.dz, kb * 64 + (j << 3));
        }
        const int rows = (is_x ? a.BH + 2 : a.BH) * Wp;         // window rows
        const int col_lo = is_x ? 1 : 0, row_off = is_x ? -1 : 0; // window column / row of image column / row 0
        const int wp0 = pos0 % Wp, hh0 = pos0 / Wp;
        const int stepq = npos / Wp, stepr = npos - stepq * Wp;
        for (int t = 0; t < my_tiles; ++t) {
            const int s = t % S, zs = t % ZS;
            const int tl = cta + t * nctas;
            const int img = tl / a.tiles_per_img, h0 = (tl - img * a.tiles_per_img) * a.BH;
            (void)img;
            if (!mbar_wait_abortable(st_full(s), (uint32_t)((t / S) & 1), abort_flag)) break;
            if (!is_x && use_z && !mbar_wait_abortable(z_full(zs), (uint32_t)((t / ZS) & 1), abort_flag)) break;
            if (need) {
                uint8_t* blk = sSt + (size_t)s * a.stage_bytes + (is_x ? (size_t)kb * a.x_block : (size_t)kbi * a.x_block + (size_t)kb * a.d_block);
                const uint8_t* zblk = sZ + (size_t)zs * a.z_bytes + (size_t)kb * a.d_block;
                int wp = wp0, hh = hh0;
#pragma unroll 4
                for (int q = pos0; q < rows; q += npos) {
                    const bool valid = wp >= col_lo && wp < col_lo + a.W && (uint32_t)(h0 + row_off + hh) < (uint32_t)a.H;
                    const uint32_t off = (uint32_t)q * 128u + (uint32_t)((j ^ (q & 7)) << 4);
                    if (valid) {
                        uint4* p = reinterpret_cast<uint4*>(blk + off);
                        *p = is_x ? xv.apply(*p) : xg.apply(*p, *reinterpret_cast<const uint4*>(zblk + off));
                    }
                    wp += stepr;
                    hh += stepq;
                    if (wp >= Wp) {
                        wp -= Wp;
                        ++hh;
                    }
                }
                fence_async_smem();
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(st_xf(s));
                if (!is_x && use_z) mbar_arrive(z_empty(zs));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: the CTA's partial
        const int q = warp & 3;
        const int k = q * 32 + lane;                             // output channel = accumulator row
        bool ok = true;
        if (my_tiles > 0) ok = mbar_wait_abortable(done, 0, abort_flag);
        fence_after_sync();
        float* pb = a.partial + (size_t)cta * a.CO * 9 * a.CI;
        for (int tt = 0; tt < t_count && ok; ++tt) {
            const int tp = t_first + tt;
            for (int g = 0; g < (a.CI >> 4); ++g) {
                float v[16];
                if (my_tiles > 0) {
                    tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(tt * a.CI + (g << 4)), v);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = 0.f;
                }
                if (k < a.CO) {
                    float* dst = pb + ((size_t)k * 9 + tp) * a.CI + (g << 4);
#pragma unroll
                    for (int hh = 0; hh < 4; ++hh) *reinterpret_cast<float4*>(dst + hh * 4) = make_float4(v[hh * 4], v[hh * 4 + 1], v[hh * 4 + 2], v[hh * 4 + 3]);
                }
            }
        }
    }
    fence_before_sync();
    __syncthreads();
    if (tid == 0 && abort_store) atomicExch(a.err, 1);
    if (warp == 1) tmem_dealloc(tmem, a.tmem_cols);
}

}  // namespace

// Returns the number of CTA partials written to `partial` ([ctas][CO][9][CI], to be summed over ctas), or 0 if the layer does not
// fit this kernel (nothing launched).
int conv3_wgrad_pipe(int n_img, int H, int W, int CI, int CO, const GradSrc& dz, const ValSrc& x, float* partial, size_t partial_floats, int* err,
                     double bytes, double flops, cudaStream_t st) {
    if (CI % 64 || CO % 64 || CI > 128 || CO > 128 || W + 2 > 126) return 0;
    if ((double)n_img * H * W * 128.0 >= 2.0e9) return 0;
    const int Wp = W + 2, kbi = CI / 64, kbo = CO / 64;
    WPArgs p{};
    p.xf_x = (x.scale != nullptr || x.act != ACT_NONE) ? 1 : 0;
    p.xf_d = grad_needs_z(dz) ? 1 : 0;
    const size_t budget = 224 * 1024;
    // the tallest tile (least halo per pixel) that leaves two (x, dy) stages and, with a transform of dy, two z stages
    bool found = false;
    for (int bh = H < 16 ? H : 16; bh >= 1 && !found; --bh) {
        if (bh * Wp > 512) continue;
        const int ksteps = (bh * Wp + 15) / 16, kpad = ksteps * 16;
        int xrows = (bh + 2) * Wp;
        if (xrows < kpad + 2 * Wp + 2) xrows = kpad + 2 * Wp + 2;  // the rows the last tap's last step reads
        const uint32_t x_block = (uint32_t)((xrows + 7) / 8 * 8) * 128u, d_block = (uint32_t)kpad * 128u;      // kpad is a multiple of 16: 1024-byte aligned
        const size_t stage = (size_t)kbi * x_block + (size_t)kbo * d_block, zb = (size_t)kbo * d_block;
        const int zs = p.xf_d ? 2 : 0;
        if (2 * stage + zs * zb > budget) continue;
        found = true;
        p.BH = bh; p.ksteps = ksteps; p.x_block = x_block; p.d_block = d_block;
        p.stage_bytes = (uint32_t)stage; p.z_bytes = (uint32_t)zb;
        p.ZS = zs;
        p.S = (int)((budget - zs * zb) / stage);
        if (p.S > WP_MAX_S) p.S = WP_MAX_S;
    }
    if (!found) return 0;
    p.x_box = 128u * (uint32_t)Wp * (uint32_t)(p.BH + 2);
    p.d_box = 128u * (uint32_t)Wp * (uint32_t)p.BH;
    p.smem_bytes = (uint32_t)p.S * p.stage_bytes + (uint32_t)p.ZS * p.z_bytes;
    if (p.ZS == 0) p.ZS = 1;
    // taps per CTA group: as many as fit the 512 accumulator columns
    int tpg = 512 / CI;
    if (tpg > 9) tpg = 9;
    const int groups = (9 + tpg - 1) / tpg;
    p.taps_per_group = (9 + groups - 1) / groups;
    p.tmem_cols = 32;
    while ((int)p.tmem_cols < p.taps_per_group * CI) p.tmem_cols <<= 1;
    p.x = x; p.dz = dz; p.partial = partial; p.err = err;
    p.n_img = n_img; p.H = H; p.W = W; p.CI = CI; p.CO = CO;
    p.tiles_per_img = (H + p.BH - 1) / p.BH;
    p.total_tiles = n_img * p.tiles_per_img;
    const size_t out_elems = (size_t)CO * 9 * CI;
    int ctas = sm_count() / groups;
    if (ctas > p.total_tiles) ctas = p.total_tiles;
    if ((size_t)ctas > partial_floats / out_elems) ctas = (int)(partial_floats / out_elems);
    if (ctas < 1) return 0;
    alignas(64) CUtensorMap mx, md, mz;
    {
        const uint64_t dx[4] = {(uint64_t)CI, (uint64_t)W, (uint64_t)H, (uint64_t)n_img};
        const uint64_t sx[3] = {(uint64_t)CI * 2, (uint64_t)W * CI * 2, (uint64_t)H * W * CI * 2};
        const uint32_t bx[4] = {64, (uint32_t)Wp, (uint32_t)(p.BH + 2), 1};
        if (!tma::encode_bf16(&mx, x.p, 4, dx, sx, bx)) return 0;
        const uint64_t dd[4] = {(uint64_t)CO, (uint64_t)W, (uint64_t)H, (uint64_t)n_img};
        const uint64_t sd[3] = {(uint64_t)CO * 2, (uint64_t)W * CO * 2, (uint64_t)H * W * CO * 2};
        const uint32_t bd[4] = {64, (uint32_t)Wp, (uint32_t)p.BH, 1};
        if (!tma::encode_bf16(&md, dz.dy, 4, dd, sd, bd)) return 0;
        if (!tma::encode_bf16(&mz, p.xf_d ? dz.z : dz.dy, 4, dd, sd, bd)) return 0;
    }
    smem_limit_once<122>(conv3_wgrad_pipe_kernel, 226 * 1024);
    // recorded bytes: the operands once and the gradient once; the per-CTA partials are the split-sum kernel's traffic
    LaunchScope ls(K_CONV3_BWD_WEIGHT_TC, bytes + 4.0 * out_elems, flops, st);
    launch_pdl(conv3_wgrad_pipe_kernel, dim3(ctas, groups), WP_THREADS, (size_t)p.smem_bytes + 1024, st, mx, md, mz, p);
    return ctas;
}

}  // namespace ast
