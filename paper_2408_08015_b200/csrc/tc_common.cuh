// tcgen05 / tensor-memory / mbarrier / bulk-copy primitives shared by the tensor-core kernels
// (inline PTX for sm_100a), and the shared-memory operand layouts they assume.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "common.cuh"

namespace ast {
namespace tc {

constexpr int TM = 128;            // rows of one MMA tile (UMMA M)
constexpr int KB = 64;             // bf16 elements per 128-byte swizzle row
constexpr uint32_t WAIT_LIMIT = 1u << 22;

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
// Bounded wait: false if the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait_limit(uint32_t mbar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(mbar, parity)) return true;
        if (i > 64) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t mbar, uint32_t parity) { return mbar_wait_limit(mbar, parity, WAIT_LIMIT); }
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

__device__ __forceinline__ void mbar_arrive(uint32_t mbar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t mbar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src), "r"(bytes), "r"(mbar)
                 : "memory");
}
// Bulk store shared -> global (one contiguous byte range; both addresses 16-byte aligned, size a
// multiple of 16) as part of the issuing thread's bulk async-group.
__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// waits until at most N of the thread's bulk groups still have to READ their shared-memory source
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
// waits until at most N of the thread's bulk groups are still incomplete
template <int N> __device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
// Named barrier over `threads` threads (a multiple of 32) that also ANDs a predicate across them.
__device__ __forceinline__ bool named_bar_and(uint32_t id, uint32_t threads, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.u32 p, %1, 0;\n"
        "bar.red.and.pred q, %2, %3, p;\n"
        "selp.u32 %0, 1, 0, q;\n"
        "}\n"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(id), "r"(threads)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ void named_bar_sync(uint32_t id, uint32_t threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }

// Bounded wait that also gives up as soon as another role has raised the abort flag.
__device__ __forceinline__ bool mbar_wait_abortable(uint32_t mbar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(mbar, parity)) return true;
        if (*abort_flag) return false;
        if (i > 32) __nanosleep(32);
    }
    *abort_flag = 1;
    return false;
}
// Issue-only forms: several loads can be in flight before one tmem_ld_wait().
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]),
          "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Pins the order: nothing that reads r[0..15] may be scheduled before this point (placed after tmem_ld_wait()).
__device__ __forceinline__ void tmem_ld_pin16(uint32_t* r) {
    asm volatile(""
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]),
                   "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])::"memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]),
          "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Issue forms for a whole warp in convergent control flow: every lane executes the instruction stream (so that the
// descriptor arithmetic can stay in the uniform datapath) and the elected lane alone issues.
__device__ __forceinline__ uint32_t elect_leader() {
    uint32_t pred;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "elect.sync _|p, 0xffffffff;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(pred));
    return pred;
}
__device__ __forceinline__ void umma_bf16_lead(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate, uint32_t leader) {
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "setp.ne.b32 q, %5, 0;\n"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(leader)
        : "memory");
}
__device__ __forceinline__ void umma_commit_lead(uint32_t mbar, uint32_t leader) {
    asm volatile(
        "{\n"
        ".reg .pred q;\n"
        "setp.ne.b32 q, %1, 0;\n"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n"
        "}\n" ::"r"(mbar),
        "r"(leader)
        : "memory");
}

// Branch-free operand transforms with per-thread register coefficients.  Absent BatchNorm
// terms take neutral values (scale 1, shift 0, k1 1, k2 = k3 0) and the activation becomes a pair
// of bounds (ReLU6: 0..6, ReLU: 0..inf, none: -inf..inf), so that every lane runs the same
// instruction stream whatever its operand.
// These transforms are bound by the integer / min-max / convert pipe (64 lanes per clock and SM, half the fused
// multiply-add pipe's rate), so they keep that pipe's work to the two unpacks and one pack per pair of elements it cannot
// avoid: the clamp of an activation is applied AFTER rounding, on packed bfloat16 pairs (rounding is monotonic and the
// bounds 0 and 6 are bfloat16 numbers, so the result is the same), and the activation mask of the backward transform is
// formed on the multiply-add pipe as a saturated product instead of a compare and a select.
struct XfVal {
    float cs[8], ch[8];
    int act;
    __device__ __forceinline__ void init(const ValSrc& s, int c0) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            cs[q] = s.scale ? __ldg(s.scale + c0 + q) : 1.f;
            ch[q] = s.scale ? __ldg(s.shift + c0 + q) : 0.f;
        }
        act = s.act;
    }
    __device__ __forceinline__ uint4 apply(const uint4& raw) const {
        Vec<__nv_bfloat16> v;
        v.raw = raw;
        float f[8];
        v.unpack(f);
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 8; q += 2) {
            const float2 r = __ffma2_rn(make_float2(f[q], f[q + 1]), make_float2(cs[q], cs[q + 1]), make_float2(ch[q], ch[q + 1]));
            __nv_bfloat162 h = __floats2bfloat162_rn(r.x, r.y);
            w[q >> 1] = *reinterpret_cast<uint32_t*>(&h);
        }
        if (act != ACT_NONE) {                      // uniform branch
            const __nv_bfloat162 zero = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                __nv_bfloat162 h = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&w[i]), zero);
                w[i] = *reinterpret_cast<uint32_t*>(&h);
            }
            if (act == ACT_RELU6) {
                const __nv_bfloat162 six = __floats2bfloat162_rn(6.f, 6.f);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    __nv_bfloat162 h = __hmin2(*reinterpret_cast<__nv_bfloat162*>(&w[i]), six);
                    w[i] = *reinterpret_cast<uint32_t*>(&h);
                }
            }
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};
// 1 for v > 0 (denormals included), 0 for v <= 0, formed on the multiply-add pipe: saturate(v * 2^126) is 1 for every
// normal positive v and at least 2^-23 for a denormal one, which the second product lifts to 1.
__device__ __forceinline__ float step_pos(float v) {
    float m;
    asm("mul.sat.f32 %0, %1, 0f7E800000;" : "=f"(m) : "f"(v));
    asm("mul.sat.f32 %0, %1, 0f7E800000;" : "=f"(m) : "f"(m));
    return m;
}
struct XfGrad {
    float cs[8], ch[8], k1[8], k2[8], k3[8];
    int act;
    __device__ __forceinline__ void init(const GradSrc& s, int c0) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            cs[q] = s.scale ? __ldg(s.scale + c0 + q) : 1.f;
            ch[q] = s.scale ? __ldg(s.shift + c0 + q) : 0.f;
            k1[q] = s.k1 ? __ldg(s.k1 + c0 + q) : 1.f;
            k2[q] = s.k1 ? __ldg(s.k2 + c0 + q) : 0.f;
            k3[q] = s.k1 ? __ldg(s.k3 + c0 + q) : 0.f;
        }
        act = s.act;
    }
    __device__ __forceinline__ uint4 apply(const uint4& rawdy, const uint4& rawz) const {
        Vec<__nv_bfloat16> v;
        float f[8], z[8];
        v.raw = rawdy;
        v.unpack(f);
        v.raw = rawz;
        v.unpack(z);
        if (act != ACT_NONE) {                      // uniform branch: dy <- dy * [pre strictly inside the linear region]
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float pre = fmaf(z[q], cs[q], ch[q]);
                float m = step_pos(pre);
                if (act == ACT_RELU6) m *= step_pos(6.f - pre);
                f[q] *= m;
            }
        }
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 8; q += 2) {
            float2 o = __ffma2_rn(make_float2(k3[q], k3[q + 1]), make_float2(z[q], z[q + 1]), make_float2(k2[q], k2[q + 1]));
            o = __ffma2_rn(make_float2(k1[q], k1[q + 1]), make_float2(f[q], f[q + 1]), o);
            __nv_bfloat162 h = __floats2bfloat162_rn(o.x, o.y);
            w[q >> 1] = *reinterpret_cast<uint32_t*>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

}  // namespace tc
}  // namespace ast
