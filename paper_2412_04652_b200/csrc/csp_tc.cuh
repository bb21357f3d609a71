// tcgen05 / tensor-memory wrappers shared by the bf16 scoring kernels.
#pragma once

#include "csp_device.cuh"

namespace csp {
namespace dev {

// ---- tcgen05 wrappers ------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// one row (TMEM lane) per thread, 32 consecutive fp32 columns
__device__ __forceinline__ void tc_ld_row32(uint32_t (&v)[32], uint32_t taddr) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
// one row (TMEM lane) per thread, 16 consecutive fp32 columns
__device__ __forceinline__ void tc_ld_row16(uint32_t (&v)[16], uint32_t taddr) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
// 16 rows x 32 columns spread over the warp like an mma accumulator: thread (lane) holds, for each
// 8-column block i, regs 4i..4i+3 = (row lane/4, cols 2(lane%4)+{0,1}), (row lane/4+8, same cols)
__device__ __forceinline__ void tc_ld_16x32(uint32_t (&v)[16], uint32_t taddr) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
// the same for 16 columns: regs 4i..4i+3 of 8-column block i = 0, 1
__device__ __forceinline__ void tc_ld_16x16(uint32_t (&v)[8], uint32_t taddr) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_frag(uint32_t (&v)[16], uint32_t taddr) { tc_ld_16x32(v, taddr); }
__device__ __forceinline__ void tc_ld_frag(uint32_t (&v)[8], uint32_t taddr) { tc_ld_16x16(v, taddr); }
// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t sw128_desc(uint32_t smem_addr) {
    uint64_t d = uint64_t((smem_addr & 0x3FFFFu) >> 4);
    d |= uint64_t(1) << 16;                // leading byte offset (unused for swizzled K-major)
    d |= uint64_t(1024 >> 4) << 32;        // stride byte offset
    d |= uint64_t(1) << 46;                // descriptor version
    d |= uint64_t(2) << 61;                // SWIZZLE_128B
    return d;
}
// three-input maximum (one instruction on sm_100)
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float lg2f(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// arrive on the mbarrier at the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_bar), "r"(rank));
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait on a barrier that CTAs of the whole cluster arrive on
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if (*abort_flag) return false;
    const unsigned long long t0 = global_ns();
    while (true) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
}

__device__ __forceinline__ float2 ex2f2(float2 x) { return make_float2(ex2f(x.x), ex2f(x.y)); }
// 2^x for two values on the FMA pipe instead of the special-function unit: x rounded to the nearest integer j
// with the 1.5 * 2^23 trick, a cubic for 2^f on f = x - j in [-0.5, 0.5] (minimax in the relative error,
// 7.5e-5), and j added to the exponent field.  x <= 126; below -125 the result stays at about 2^-125.
__device__ __forceinline__ float2 ex2_fma2(float2 x) {
    x = make_float2(fmaxf(x.x, -125.f), fmaxf(x.y, -125.f));
    const float2 t = __fadd2_rn(x, make_float2(12582912.f, 12582912.f));
    const float2 j = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
    const float2 f = __ffma2_rn(j, make_float2(-1.f, -1.f), x);
    float2 p = __ffma2_rn(make_float2(0.0551716648f, 0.0551716648f), f, make_float2(0.2426111251f, 0.2426111251f));
    p = __ffma2_rn(p, f, make_float2(0.6932609677f, 0.6932609677f));
    p = __ffma2_rn(p, f, make_float2(0.9999280572f, 0.9999280572f));
    return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),
                       __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}

// ---- pass-1 row statistics of one accumulator block of 32 rows x 8 NB columns ----------------------------
// v0 / v1: the two 16-row halves as loaded by tc_ld_frag.  Statistic slot jj = 2 nt + e belongs to column
// 8 nt + 2 (lane % 4) + e of the block; (m, z) is a running (reference, sum of 2^(x scale2 - reference)) over
// the keys this thread has seen.  The reference is only raised when a value exceeds it by more than kLazy,
// which is rare after the first tiles: the test is taken once for the whole block, so that the exponentials
// that follow are straight-line code.  scale2 > 0.
// kFma: one pair of exponentials in eight goes to the FMA pipe (kernels bound by the special-function unit).
template <int NB, bool kFma = false>
__device__ __forceinline__ void stats_block(const uint32_t (&v0)[4 * NB], const uint32_t (&v1)[4 * NB],
                                            float (&m)[2 * NB], float (&z)[2 * NB], float scale2) {
    float mx[2 * NB];       // largest raw value of the slot (scale2 > 0: scaling keeps the order)
    bool raise = false;
#pragma unroll
    for (int jj = 0; jj < 2 * NB; ++jj) {
        const int i = (jj >> 1) * 4 + (jj & 1);
        mx[jj] = fmax3(__uint_as_float(v0[i]), __uint_as_float(v0[i + 2]),
                       fmaxf(__uint_as_float(v1[i]), __uint_as_float(v1[i + 2])));
        raise |= fmaf(mx[jj], scale2, -m[jj]) > kLazy;
    }
    if (raise) {
#pragma unroll
        for (int jj = 0; jj < 2 * NB; ++jj) {
            const float ms = mx[jj] * scale2;
            if (ms > m[jj] + kLazy) { z[jj] *= ex2f(m[jj] - ms); m[jj] = ms; }
        }
    }
    // Slots 2 b and 2 b + 1 sit in neighbouring registers of every fragment, so the scaling and the sums run
    // as two-wide fp32 instructions (same roundings and summation order as the scalar form, half the
    // instructions to issue).
    const float2 sc2 = make_float2(scale2, scale2);
#pragma unroll
    for (int bq = 0; bq < NB; ++bq) {
        const float2 nm = make_float2(-m[2 * bq], -m[2 * bq + 1]);
        const float2 ea = ex2f2(__ffma2_rn(make_float2(__uint_as_float(v0[4 * bq]), __uint_as_float(v0[4 * bq + 1])), sc2, nm));
        const float2 eb = ex2f2(__ffma2_rn(make_float2(__uint_as_float(v0[4 * bq + 2]), __uint_as_float(v0[4 * bq + 3])), sc2, nm));
        const float2 ec = ex2f2(__ffma2_rn(make_float2(__uint_as_float(v1[4 * bq]), __uint_as_float(v1[4 * bq + 1])), sc2, nm));
        const float2 xd = __ffma2_rn(make_float2(__uint_as_float(v1[4 * bq + 2]), __uint_as_float(v1[4 * bq + 3])), sc2, nm);
        const float2 ed = (kFma && (bq & 1)) ? ex2_fma2(xd) : ex2f2(xd);
        const float2 zz = __fadd2_rn(make_float2(z[2 * bq], z[2 * bq + 1]), __fadd2_rn(__fadd2_rn(ea, eb), __fadd2_rn(ec, ed)));
        z[2 * bq] = zz.x;
        z[2 * bq + 1] = zz.y;
    }
}
// The same for a tile that reaches into the window: key t is visible to window column w iff w < W and
// t <= first_masked_key + w.  t_base = key of this thread's first row; col0 = window column of the block's
// first column plus 2 (lane % 4).
template <int NB>
__device__ __forceinline__ void stats_block_masked(const uint32_t (&v0)[4 * NB], const uint32_t (&v1)[4 * NB],
                                                   float (&m)[2 * NB], float (&z)[2 * NB], float scale2, int t_base,
                                                   int first_masked_key, int W, int col0) {
#pragma unroll
    for (int jj = 0; jj < 2 * NB; ++jj) {
        const int i = (jj >> 1) * 4 + (jj & 1);
        const int colw = col0 + (jj >> 1) * 8 + (jj & 1);
        float x[4] = {__uint_as_float(v0[i]) * scale2, __uint_as_float(v0[i + 2]) * scale2,
                      __uint_as_float(v1[i]) * scale2, __uint_as_float(v1[i + 2]) * scale2};
        bool vis[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int t = t_base + (r & 1) * 8 + (r >> 1) * 16;
            vis[r] = colw < W && t <= first_masked_key + colw;
            x[r] = vis[r] ? x[r] : kNeg;
        }
        const float mx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
        if (mx > m[jj] + kLazy) { z[jj] *= ex2f(m[jj] - mx); m[jj] = mx; }
        const float mm = m[jj];
#pragma unroll
        for (int r = 0; r < 4; ++r) z[jj] += vis[r] ? ex2f(x[r] - mm) : 0.f;
    }
}

}  // namespace dev
}  // namespace csp
