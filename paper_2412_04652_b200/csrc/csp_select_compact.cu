// Selection and compaction in one persistent kernel (Eq. 2-4) for launches with many short units.
//
// The selection of a unit is a chain of short dependent phases (histogram, barrier, bin walk) that leaves the
// memory system idle; the compaction is pure data movement.  Run one after the other, the first costs a fifth
// of the second's time.  Here one CTA per SM walks over units blockIdx.x, blockIdx.x + gridDim.x, ... with
// its warps split by role, so that the selection of later units hides under the copy of earlier ones:
//   warps 0-15   selection team: sel::select_unit on one unit after the other, as far ahead as it likes (its
//                results go to global memory: keep_idx, n_out, and the labels of the kept positions, which it holds
//                in registers); after each unit it publishes a counter
//   next 4 (3)   gather team: for every kept row, 16-byte asynchronous copies (cp.async) from the row's place in
//                K and V into a stage of shared memory, where the kept rows of a unit lie back to back
//   last warp    store: one bulk copy (cp.async.bulk) per tensor and stage from shared memory to the output,
//                where kept rows are contiguous as well
// No register staging: what is in flight is bounded by shared memory (six stages of 32 KB, or eight of 24 KB with
// three gather warps), not by the register file.  Stages of 16 KB were 13 % slower on the copy, stages of 64 KB 2 %;
// 24 and 32 KB are level, and so are 3, 4 and 8 gather warps.  A warp of its own for the labels (two dependent loads per
// kept row) cost registers the selection needs, and fetching them in the gather team held every stage up (the copy took
// twice as long): the selection team has them in registers.  Every wait is bounded.
//
// Preconditions (checked by the launcher): the longest cache has at most 8192 positions (16 keys per selection
// thread), the outputs are a second, dense buffer with contiguous rows, the cache is not paged.
#include "csp_select_unit.cuh"

namespace csp {
namespace {
using namespace dev;

constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kAhead = 2;                                // stages between the fetch of a row's position and its use
constexpr int kStoresPending = 2;                        // bulk stores that may still be reading shared memory
constexpr int kMaxStages = 8;

// The CTA's shape follows from the registers the selection needs.  The register file is four partitions of 16384
// registers, each holding a quarter of the CTA's warps: 21 warps (four of them gathering) may use 80 registers a thread,
// which 4 or 8 keys per selection thread fit; 16 keys need 96, which leaves room for 20 warps (three gathering).
template <int E>
struct Shape {
    static constexpr int kGatherWarps = E > 8 ? 3 : 4;
    static constexpr int kGatherThreads = 32 * kGatherWarps;
    static constexpr int kStoreWarp = kSelWarps + kGatherWarps;
    static constexpr int kThreads = kSelThreads + kGatherThreads + 32;
    static constexpr int kRegisters = E > 8 ? 96 : 80;
    static constexpr int kHalfStage = E > 8 ? 12288 : 16384;          // bytes of K (and of V) per stage
    static constexpr int kStageBytes = 2 * kHalfStage;
    static constexpr int kChunksPerThread = kHalfStage / 16 / kGatherThreads;   // 16-byte chunks of one tensor per gather thread and stage
    static constexpr int kStages = E > 8 ? 8 : 6;
    static constexpr int kDepth = E > 8 ? 4 : 3;                      // stages a gather thread keeps in flight
    static_assert((kThreads / 32 + 3) / 4 * (kRegisters * 32) <= 16384, "the CTA must fit the register file");
    static_assert(kStages >= kDepth + kStoresPending + 1 && kStages <= kMaxStages, "ring too short for the copies in flight");
    static_assert(kChunksPerThread * kGatherThreads * 16 == kHalfStage, "stage must divide among the gather threads");
};

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void st_shared_zero16(uint32_t dst) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0u) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void st_release_shared(uint32_t addr, int v) {
    asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_shared(uint32_t addr) {
    int v;
    asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}

// Waits until the selection team has finished `want` units; false (and the abort flag raised) if that takes too long.
__device__ __forceinline__ bool wait_selected(uint32_t counter, int want, volatile int* abort_flag) {
    if (ld_acquire_shared(counter) >= want) return true;
    const unsigned long long t0 = global_ns();
    while (true) {
        __nanosleep(100);                                // the selection team needs the issue slots more than this loop
        if (ld_acquire_shared(counter) >= want) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
}

template <int E, int CPR>    // keys per selection thread (4, 8 or 16); 16-byte chunks per row (8, 16 or 32)
__global__ void __maxnreg__(Shape<E>::kRegisters)
select_compact_kernel(const SelectArgs sa, const CompactArgs ca, const int n_units) {
    using S = Shape<E>;
    constexpr int kGatherThreads = S::kGatherThreads, kStoreWarp = S::kStoreWarp, kHalfStage = S::kHalfStage;
    constexpr int kStageBytes = S::kStageBytes, kChunksPerThread = S::kChunksPerThread, kDepth = S::kDepth;
    constexpr int n_stages = S::kStages;
    constexpr int kRowsPerStage = kHalfStage / (16 * CPR);
    constexpr int kRowStep = kGatherThreads / CPR;       // rows between two chunks of one gather thread
    static_assert(kGatherThreads % CPR == 0, "whole rows per pass of the gather team");
    __shared__ sel::SelectSmem<kSelWarps> sm;
    __shared__ __align__(8) uint64_t bars[2 * kMaxStages];
    __shared__ int selected;                             // units the selection team has finished
    __shared__ int abort_word;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t stage0 = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t full = smem_u32(&bars[0]), empty = smem_u32(&bars[kMaxStages]);
    const uint32_t counter = smem_u32(&selected);
    volatile int* const abort_flag = &abort_word;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        selected = 0;
        abort_word = 0;
        for (int s = 0; s < n_stages; ++s) { mbar_init(full + 8 * s, kGatherThreads); mbar_init(empty + 8 * s, 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp < kSelWarps) {
        // =============================== selection team ===============================
        int done = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            sel::select_unit<kSelThreads, E, true>(sa, u, sm, (ca.mod_out && ca.modality) ? ca.mod_out : nullptr);
            // keep_idx and n_out of this unit are written: order them before the counter, and keep the next
            // unit's writes to the team's shared memory behind this unit's last reads
            __threadfence();
            asm volatile("bar.sync %0, %1;" ::"n"(sel::kTeamBarrier), "n"(kSelThreads) : "memory");
            ++done;
            if (tid == 0) st_release_shared(counter, done);
        }
    } else if (warp < kStoreWarp) {
        // =============================== gather team ===============================
        const int g = tid - kSelThreads;
        const int r_in = g / CPR, c = g % CPR;
        const uint4* const kin = static_cast<const uint4*>(ca.k);
        const uint4* const vin = static_cast<const uint4*>(ca.v);
        int issued = 0, arrived = 0;                     // stages this thread has committed / signalled as complete
        // every stage whose copies have landed is fenced towards the bulk-copy engine and signalled
        auto signal_upto = [&](int upto) {
            if (arrived < upto) fence_async_smem();
            for (; arrived < upto; ++arrived) mbar_arrive(full + 8 * (arrived % n_stages));
        };
        int j = 0;
        for (int u = blockIdx.x; u < n_units && !*abort_flag; u += gridDim.x, ++j) {
            if (ld_acquire_shared(counter) <= j) {       // nothing to do yet: let what is in flight go out meanwhile
                cp_async_wait<0>();
                signal_upto(issued);
                if (!wait_selected(counter, j + 1, abort_flag)) break;
            }
            const int b = u / ca.n_kv_heads, h = u % ca.n_kv_heads;
            int n = __ldcg(ca.n_out + u);
            if (n > ca.out_capacity) n = ca.out_capacity;           // the selection has flagged it already
            if (n <= 0) continue;
            const int32_t* const idx = ca.keep_idx + int64_t(u) * ca.out_capacity;
            const int64_t kbase = int64_t(b) * ca.k_sb + int64_t(h) * ca.k_sh + c;
            const int64_t vbase = int64_t(b) * ca.v_sb + int64_t(h) * ca.v_sh + c;
            // positions of this thread's rows, fetched kAhead stages before their use (a load from L2 under full
            // memory load takes longer than one stage lasts)
            int t_q[kAhead][kChunksPerThread];
#pragma unroll
            for (int s_ = 0; s_ < kAhead; ++s_)
#pragma unroll
                for (int q = 0; q < kChunksPerThread; ++q) {
                    const int row = s_ * kRowsPerStage + q * kRowStep + r_in;
                    t_q[s_][q] = row < n ? __ldcg(idx + row) : -1;
                }
            for (int r0 = 0; r0 < n; r0 += kRowsPerStage, ++issued) {
                int t_cur[kChunksPerThread];
#pragma unroll
                for (int q = 0; q < kChunksPerThread; ++q) {
                    t_cur[q] = t_q[0][q];
#pragma unroll
                    for (int s_ = 0; s_ + 1 < kAhead; ++s_) t_q[s_][q] = t_q[s_ + 1][q];
                    const int row = r0 + kAhead * kRowsPerStage + q * kRowStep + r_in;
                    t_q[kAhead - 1][q] = row < n ? __ldcg(idx + row) : -1;
                }
                const int slot = issued % n_stages;
                mbar_wait(empty + 8 * slot, (uint32_t(issued / n_stages) & 1u) ^ 1u, abort_flag);
                if (*abort_flag) break;
                const uint32_t dst = stage0 + uint32_t(slot) * kStageBytes + uint32_t(g) * 16u;
#pragma unroll
                for (int q = 0; q < kChunksPerThread; ++q) {
                    const int t = t_cur[q];
                    if (t >= 0 && t < ca.max_len) {
                        cp_async_16(dst + uint32_t(q) * (kGatherThreads * 16u), kin + kbase + int64_t(t) * ca.k_st);
                        cp_async_16(dst + kHalfStage + uint32_t(q) * (kGatherThreads * 16u), vin + vbase + int64_t(t) * ca.v_st);
                    } else if (t >= 0) {                 // an index outside the cache (never the selection's own): zeros
                        st_shared_zero16(dst + uint32_t(q) * (kGatherThreads * 16u));
                        st_shared_zero16(dst + kHalfStage + uint32_t(q) * (kGatherThreads * 16u));
                    }
                }
                cp_async_commit();
                if (issued + 1 - arrived >= kDepth) {    // the oldest stage in flight has had the longest to land
                    cp_async_wait<kDepth - 1>();
                    signal_upto(issued + 1 - (kDepth - 1));
                }
            }
        }
        cp_async_wait<0>();                              // also on the way out after a timeout: nothing may land later
        signal_upto(issued);
    } else if (lane == 0) {
        // =============================== store ===============================
        uint8_t* const kout = static_cast<uint8_t*>(ca.k_out);
        uint8_t* const vout = static_cast<uint8_t*>(ca.v_out);
        int stored = 0, released = 0;
        int j = 0;
        for (int u = blockIdx.x; u < n_units && !*abort_flag; u += gridDim.x, ++j) {
            if (!wait_selected(counter, j + 1, abort_flag)) break;
            const int b = u / ca.n_kv_heads, h = u % ca.n_kv_heads;
            int n = __ldcg(ca.n_out + u);
            if (n > ca.out_capacity) n = ca.out_capacity;
            if (n <= 0) continue;
            uint8_t* const ko = kout + (int64_t(b) * ca.ko_sb + int64_t(h) * ca.ko_sh) * 16;
            uint8_t* const vo = vout + (int64_t(b) * ca.vo_sb + int64_t(h) * ca.vo_sh) * 16;
            for (int r0 = 0; r0 < n; r0 += kRowsPerStage, ++stored) {
                const int slot = stored % n_stages;
                mbar_wait(full + 8 * slot, uint32_t(stored / n_stages) & 1u, abort_flag);
                if (*abort_flag) break;
                fence_async_smem();
                const int rows = min(kRowsPerStage, n - r0);
                const uint32_t src = stage0 + uint32_t(slot) * kStageBytes;
                bulk_store(ko + int64_t(r0) * (CPR * 16), src, uint32_t(rows) * (CPR * 16));
                bulk_store(vo + int64_t(r0) * (CPR * 16), src + kHalfStage, uint32_t(rows) * (CPR * 16));
                bulk_commit();
                // a stage goes back to the gather team once its stores have read it
                if (stored + 1 - released > kStoresPending) {
                    bulk_wait_read<kStoresPending>();
                    for (; released < stored + 1 - kStoresPending; ++released) mbar_arrive(empty + 8 * (released % n_stages));
                }
            }
        }
        bulk_wait_all();                                 // the outputs are complete when the kernel ends
        if (*abort_flag) atomicOr(ca.status, CSP_DEV_TIMEOUT);
    }
    __syncthreads();                                     // shared memory stays until every copy has been waited for
}

}  // namespace

// Launches the fused kernel if the shape qualifies; *taken tells whether it did.
csp_status launch_select_compact(const csp_params& p, const SelectArgs& sa, const CompactArgs& ca, cudaStream_t s,
                                 bool* taken) {
    *taken = false;
    const int units = p.batch * p.n_kv_heads;
    const int sms = sm_count();
    // Measured against the two kernels one after the other (d = 128, a quarter of the rows kept): 4 % faster with 160
    // units of 4096 positions, 9 % with 256, 15 % with 1024; 13 % faster at 2048 positions, 9 % at 1500, even at 1024,
    // slower at 512.  With 16 keys per selection thread (above 4096 positions): 10 % faster with 1024 units of 8192
    // positions (2080 rows kept), 6 % with 512, even with 320, 2 % slower with 256.
    if (units < sms || p.out_capacity == 0) return CSP_OK;
    if (p.max_len <= 1024 || p.max_len > 8192) return CSP_OK;           // one 512-thread team per unit, 4, 8 or 16 keys a thread
    // with 16 keys per thread one team selects a unit in about 22 us: the copy of a unit must be at least as long for the
    // selection to hide (a ragged batch of 1024 units of up to 8109 positions: 5 % slower when 405 rows are kept per unit,
    // 5 % faster with 811, 12 % with 1622 and 3244)
    if (p.max_len > 4096 && (units < 2 * sms || int64_t(p.out_capacity) * 12 < p.max_len)) return CSP_OK;
    if (ca.page_table || !ca.status) return CSP_OK;
    if (ca.k == ca.k_out || ca.v == ca.v_out) return CSP_OK;
    if (ca.ko_st != ca.chunks_per_row || ca.vo_st != ca.chunks_per_row) return CSP_OK;   // kept rows back to back
    auto go = [&](auto kern, auto shape, std::atomic<bool> (&configured)[kMaxDevices]) {
        using S = decltype(shape);
        const size_t smem = size_t(S::kStages) * S::kStageBytes + 128;
        if (!raise_smem_limit(kern, int(smem), configured)) return CSP_ERR_CUDA;
        kern<<<sms, S::kThreads, smem, s>>>(sa, ca, units);
        if (cudaGetLastError() != cudaSuccess) return CSP_ERR_CUDA;
        *taken = true;
        return CSP_OK;
    };
    static std::atomic<bool> cfg[9][kMaxDevices];
    const int e = p.max_len > 4096 ? 16 : (p.max_len > 2048 ? 8 : 4);
    switch (ca.chunks_per_row) {
        case 8:
            return e == 16 ? go(select_compact_kernel<16, 8>, Shape<16>(), cfg[0])
                 : e == 8  ? go(select_compact_kernel<8, 8>, Shape<8>(), cfg[1]) : go(select_compact_kernel<4, 8>, Shape<4>(), cfg[2]);
        case 16:
            return e == 16 ? go(select_compact_kernel<16, 16>, Shape<16>(), cfg[3])
                 : e == 8  ? go(select_compact_kernel<8, 16>, Shape<8>(), cfg[4]) : go(select_compact_kernel<4, 16>, Shape<4>(), cfg[5]);
        case 32:
            return e == 16 ? go(select_compact_kernel<16, 32>, Shape<16>(), cfg[6])
                 : e == 8  ? go(select_compact_kernel<8, 32>, Shape<8>(), cfg[7]) : go(select_compact_kernel<4, 32>, Shape<4>(), cfg[8]);
        default: return CSP_OK;
    }
}

}  // namespace csp
