// Pointwise (1x1, stride 1) convolution, forward and backward-data, for layers with more than 256 channels
// on one side (which the pointwise pipeline of pw_tc.cu cannot keep resident): a persistent warp-specialised
// GEMM whose reduction streams through shared memory in 64-channel blocks.
//
//   out[p][n] = sum_k A[p][k] * W[n][k]      A = act(x*scale + shift) (forward) or the BatchNorm-backward
//                                            transform of (dy, z) (backward-data), W = [N][K] bf16
//
// A tile is 128 consecutive pixels.  One 64-channel block of it arrives by ONE 2-D tensor copy, already in
// the swizzled K-major layout the MMA reads, and is transformed IN PLACE; the ring of such blocks is the only
// operand staging there is, so the whole reduction never has to be resident.  The weights of the CTA's NC
// output channels (64 or 128; wider layers are split over CTAs by output channel) stay resident for all
// blocks.  Roles as in the 3x3 pipeline (conv3_pipe.cu):
//
//   warp 0        producer: per (tile, channel block) one tensor copy of the raw block (and of z, second ring)
//   warps 1-2     MMA issuers, alternating tiles, each into its own accumulator set: 4 tcgen05.mma per block
//   warps 3-14    transform in place (all warps on the same block)
//   warps 15-18   epilogue: tcgen05.ld, (+ residual gradient), round to bf16, 16-byte stores
//
// Every warp of a role observes every block's barrier phases in order and acknowledges them.  Every wait is
// bounded and reports through the error word.
#include <cuda_bf16.h>

#include "kernels.h"
#include "tc_common.cuh"
#include "tma.cuh"

namespace ast {
namespace {

using namespace tc;
constexpr int PS_XF_WARPS = 12, PS_EPI_WARPS = 4, PS_MMA_WARPS = 2;
constexpr int PS_FIRST_XF = 1 + PS_MMA_WARPS;
constexpr int PS_THREADS = (PS_FIRST_XF + PS_XF_WARPS + PS_EPI_WARPS) * 32;
constexpr int PS_MAX_S = 6, PS_MAX_ZS = 3;
constexpr uint32_t PS_SLOT = TM * 128u;        // bytes of one 64-channel block of a tile

struct PSArgs {
    ValSrc x;                  // forward: coefficient pointers and activation (data come through the tensor map)
    GradSrc dz;                // backward: likewise
    const void* addend;        // backward only, may be null: [P][N]
    __nv_bfloat16* out;        // [P][N]
    int* err;
    int P, K, N;               // pixels, reduction channels (multiple of 64), output channels (multiple of NC)
    int NC;                    // output channels per CTA: 64 or 128
    int tiles, n_split;
    int S, ZS;                 // ring depths: operand blocks, z blocks
    int need_xf;
};

template <bool BWD>
__global__ void __launch_bounds__(PS_THREADS, 1)
pw_stream_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_z, const __grid_constant__ CUtensorMap tm_w,
                 const PSArgs a) {
    pdl_launch();
    extern __shared__ uint8_t smem_raw[];
    // w_full, slot_full[S], slot_xf[S], slot_empty[S], z_full[ZS], z_empty[ZS], acc_full[2], acc_empty[2]
    __shared__ uint64_t bars[1 + 3 * PS_MAX_S + 2 * PS_MAX_ZS + 4];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_store;
    volatile int* abort_flag = &abort_store;
    uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kbs = a.K >> 6, S = a.S, ZS = a.ZS, NC = a.NC;
    const uint32_t wblock = (uint32_t)NC * 128u;           // bytes of the resident weights of one channel block
    const uint32_t wbytes = (uint32_t)kbs * wblock;
    uint8_t* sB = base;
    uint8_t* sA = sB + wbytes;
    uint8_t* sZ = sA + (size_t)S * PS_SLOT;
    const bool use_z = BWD && a.need_xf;
    const uint32_t bar0 = smem_u32(&bars[0]);
    auto w_full = [&]() { return bar0; };
    auto slot_full = [&](int s) { return bar0 + 8u * (1 + s); };
    auto slot_xf = [&](int s) { return bar0 + 8u * (1 + PS_MAX_S + s); };
    auto slot_empty = [&](int s) { return bar0 + 8u * (1 + 2 * PS_MAX_S + s); };
    auto z_full = [&](int s) { return bar0 + 8u * (1 + 3 * PS_MAX_S + s); };
    auto z_empty = [&](int s) { return bar0 + 8u * (1 + 3 * PS_MAX_S + PS_MAX_ZS + s); };
    auto acc_full = [&](int s) { return bar0 + 8u * (1 + 3 * PS_MAX_S + 2 * PS_MAX_ZS + s); };
    auto acc_empty = [&](int s) { return bar0 + 8u * (1 + 3 * PS_MAX_S + 2 * PS_MAX_ZS + 2 + s); };
    const int half = blockIdx.x % a.n_split, n0 = half * NC;
    const int cta = blockIdx.x / a.n_split, nctas = gridDim.x / a.n_split;
    const int my_tiles = cta < a.tiles ? (a.tiles - cta + nctas - 1) / nctas : 0;
    const int total_items = my_tiles * kbs;
    const uint32_t tmem_cols = NC == 128 ? 256u : 128u;

    if (tid == 0) {
        mbar_init(w_full(), 1);
        for (int s = 0; s < PS_MAX_S; ++s) {
            mbar_init(slot_full(s), 1);
            mbar_init(slot_xf(s), PS_XF_WARPS);
            mbar_init(slot_empty(s), PS_MMA_WARPS);
        }
        for (int s = 0; s < PS_MAX_ZS; ++s) {
            mbar_init(z_full(s), 1);
            mbar_init(z_empty(s), PS_XF_WARPS);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(acc_full(s), 1);
            mbar_init(acc_empty(s), PS_EPI_WARPS);
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
        // the weights are written only by the refresh kernel, which never releases its dependents early: safe before the wait
        tma::prefetch_map(&tm_w);
        tma::prefetch_map(&tm_a);
        mbar_expect_tx(w_full(), wbytes);
        for (int kb = 0; kb < kbs; ++kb) tma::load_2d(smem_u32(sB) + (uint32_t)kb * wblock, &tm_w, kb * 64, n0, w_full());
    }
    pdl_wait();
    const uint32_t tmem = tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            int it = 0, zit = 0;
            bool ok = true;
            for (int t = 0; t < my_tiles && ok; ++t) {
                const int p0 = (cta + t * nctas) * TM;
                for (int kb = 0; kb < kbs; ++kb) {
                    const int s = it % S, n = it / S;
                    if (n > 0 && !mbar_wait_abortable(slot_empty(s), (uint32_t)((n - 1) & 1), abort_flag)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(slot_full(s), PS_SLOT);
                    tma::load_2d(smem_u32(sA + (size_t)s * PS_SLOT), &tm_a, kb * 64, p0, slot_full(s));
                    if (use_z) {
                        const int zs = it % ZS, zn = it / ZS;
                        if (zn > 0 && !mbar_wait_abortable(z_empty(zs), (uint32_t)((zn - 1) & 1), abort_flag)) {
                            ++it;      // the operand copy of this block is in flight: the drain below waits for it
                            ok = false;
                            break;
                        }
                        mbar_expect_tx(z_full(zs), PS_SLOT);
                        tma::load_2d(smem_u32(sZ + (size_t)zs * PS_SLOT), &tm_z, kb * 64, p0, z_full(zs));
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
    } else if (warp < PS_FIRST_XF) {
        // ------------------------------------------------------------ MMA issuers: warp w takes tiles w-1, w+1, ...
        const int iss = warp - 1;
        const uint32_t leader = elect_leader();
        const uint32_t idesc = make_idesc(NC);
        const uint64_t dconst = make_desc(0);
        const uint32_t b0 = smem_u32(sB) >> 4;
        bool ok = mbar_wait_abortable(w_full(), 0, abort_flag);
        for (int it = 0; it < total_items && ok; ++it) {
            const int t = it / kbs, kb = it - t * kbs;
            const bool mine = (t % PS_MMA_WARPS) == iss;
            const int s = it % S, b = t & 1, n = t >> 1;
            if (mine && kb == 0 && n > 0 && !mbar_wait_abortable(acc_empty(b), (uint32_t)((n - 1) & 1), abort_flag)) break;
            if (!mbar_wait_abortable(slot_xf(s), (uint32_t)((it / S) & 1), abort_flag)) break;
            if (mine) {
                fence_after_sync();
                const uint32_t ar = smem_u32(sA + (size_t)s * PS_SLOT) >> 4;
                const uint32_t br = b0 + (uint32_t)kb * (wblock >> 4);
                const uint32_t d = tmem + (uint32_t)(b * NC);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_bf16_lead(d, dconst + (uint64_t)(ar + 2u * ks), dconst + (uint64_t)(br + 2u * ks), idesc, (kb > 0 || ks > 0) ? 1u : 0u, leader);
                umma_commit_lead(slot_empty(s), leader);
                if (kb == kbs - 1) umma_commit_lead(acc_full(b), leader);
            } else if (leader) {
                mbar_arrive(slot_empty(s));
            }
            __syncwarp();
        }
    } else if (warp < PS_FIRST_XF + PS_XF_WARPS) {
        // ------------------------------------------------------------ transform (in place)
        // thread (pos0, j) owns 16-byte chunk j of rows pos0, pos0 + 48, pos0 + 96 of every block
        const int xt = tid - PS_FIRST_XF * 32;
        const int j = xt & 7, pos0 = xt >> 3;
        constexpr int NPOS = PS_XF_WARPS * 4, NI = (TM + NPOS - 1) / NPOS;
        // 48 rows are a multiple of 8: the swizzle term of a thread's chunk is the same in all its rows
        const uint32_t off0 = (uint32_t)pos0 * 128u + (uint32_t)((j ^ (pos0 & 7)) << 4);
        XfVal xv;
        XfGrad xg;
        for (int it = 0; it < total_items; ++it) {
            const int s = it % S, zs = it % ZS;
            const int t = it / kbs, kb = it - t * kbs;
            const int rows_left = a.P - (cta + t * nctas) * TM;      // rows past the end of the tensor were delivered as zeros and stay zeros
            if (a.need_xf && (kbs > 1 || it == 0)) {                  // the channel block changes from item to item
                if (BWD) xg.init(a.dz, kb * 64 + (j << 3));
                else xv.init(a.x, kb * 64 + (j << 3));
            }
            if (!mbar_wait_abortable(slot_full(s), (uint32_t)((it / S) & 1), abort_flag)) break;
            if (use_z && !mbar_wait_abortable(z_full(zs), (uint32_t)((it / ZS) & 1), abort_flag)) break;
            if (a.need_xf) {
                uint8_t* slot = sA + (size_t)s * PS_SLOT + off0;
                const uint8_t* zslot = sZ + (size_t)zs * PS_SLOT + off0;
#pragma unroll
                for (int i = 0; i < NI; ++i) {
                    const int q = pos0 + NPOS * i;
                    if (q < TM && q < rows_left) {
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
            const int p = (cta + t * nctas) * TM + q * 32 + lane;
            if (!mbar_wait_abortable(acc_full(b), (uint32_t)(n & 1), abort_flag)) break;
            fence_after_sync();
            for (int c0 = 0; c0 < NC; c0 += 64) {
                uint32_t rr[4][16];
#pragma unroll
                for (int u = 0; u < 4; ++u) tmem_ld16_issue(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * NC + c0 + (u << 4)), rr[u]);
                tmem_ld_wait();
#pragma unroll
                for (int u = 0; u < 4; ++u) tmem_ld_pin16(rr[u]);
                if (p < a.P) {
                    const size_t e0 = (size_t)p * a.N + n0 + c0;
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

}  // namespace

// Forward (bwd == false: x [P][K], w = [N][K]) or backward-data (bwd == true: dz [P][K] with K = c_out, w = [N][K] with N = c_in)
// through the streaming kernel.  Returns false (nothing launched) if the layer does not fit it.
bool pw_stream(bool bwd, int P, int K, int N, const ValSrc& x, const GradSrc& dz, const __nv_bfloat16* w, const void* addend, void* out, int* err,
               int kind, double bytes, cudaStream_t st) {
    if (K % 64 || N % 64 || P < 1 || (double)P * (K > N ? K : N) >= 2.0e9) return false;
    PSArgs p{};
    const int kbs = K / 64;
    const size_t budget = 225 * 1024 - 1024;
    const bool need_xf = bwd ? grad_needs_z(dz) : (x.scale != nullptr || x.act != ACT_NONE);
    const bool zring = bwd && need_xf;
    // 128 output channels per CTA where their resident weights leave room for the rings, else 64
    p.NC = 0;
    for (int nc = 128; nc >= 64 && !p.NC; nc >>= 1) {
        if (N % nc) continue;
        const size_t wbytes = (size_t)kbs * nc * 128;
        const size_t need = wbytes + (size_t)(zring ? 3 + 2 : 3) * PS_SLOT;
        if (need <= budget) {
            p.NC = nc;
            size_t left = (budget - wbytes) / PS_SLOT;
            p.ZS = zring ? (left >= 8 ? 3 : 2) : 1;
            p.S = (int)left - (zring ? p.ZS : 0);
            if (p.S > PS_MAX_S) p.S = PS_MAX_S;
        }
    }
    if (!p.NC) return false;
    p.x = x; p.dz = dz; p.addend = addend; p.out = (__nv_bfloat16*)out; p.err = err;
    p.P = P; p.K = K; p.N = N; p.tiles = (P + TM - 1) / TM; p.n_split = N / p.NC; p.need_xf = need_xf ? 1 : 0;
    alignas(64) CUtensorMap ma, mz, mw;
    {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)P};
        const uint64_t strides[1] = {(uint64_t)K * 2};
        const uint32_t box[2] = {64, TM};
        if (!tma::encode_bf16(&ma, bwd ? dz.dy : x.p, 2, dims, strides, box)) return false;
        if (!tma::encode_bf16(&mz, zring ? dz.z : (bwd ? dz.dy : x.p), 2, dims, strides, box)) return false;
        const uint64_t wd[2] = {(uint64_t)K, (uint64_t)N};
        const uint32_t wb[2] = {64, (uint32_t)p.NC};
        if (!tma::encode_bf16(&mw, w, 2, wd, strides, wb)) return false;
    }
    const size_t smem = (size_t)kbs * p.NC * 128 + (size_t)(p.S + (zring ? p.ZS : 0)) * PS_SLOT + 1024;
    smem_limit_once<123>(pw_stream_kernel<false>, 226 * 1024);
    smem_limit_once<124>(pw_stream_kernel<true>, 226 * 1024);
    int nctas = sm_count() / p.n_split;
    if (nctas < 1) nctas = 1;
    if (nctas > p.tiles) nctas = p.tiles;
    LaunchScope ls(kind, bytes, 2.0 * P * (double)N * K, st);
    if (bwd) launch_pdl(pw_stream_kernel<true>, nctas * p.n_split, PS_THREADS, smem, st, ma, mz, mw, p);
    else launch_pdl(pw_stream_kernel<false>, nctas * p.n_split, PS_THREADS, smem, st, ma, mz, mw, p);
    return true;
}

}  // namespace ast
