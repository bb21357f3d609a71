// One unit of the selection (Eq. 2-3 and the index side of Eq. 4) as a device function, shared by the
// stand-alone selection kernel (a cluster of CTAs per unit) and by the fused selection + compaction kernel
// (a team of warps inside a persistent CTA, one unit after the other).
//
// Every thread keeps E (4 or 8 or 16) of the unit's keys in registers for the whole unit (the
// order-preserving integer images of both scores plus a label bit); a warp covers 32 E consecutive
// positions, lane l holding positions base + 32 e + l, so loads are coalesced and "position order" inside
// a warp is (e, lane) order, which ballots enumerate for free.
//
// Up to four top-K problems run together (intra/inter score x text/visual keys, or intra/inter
// over all keys).  An MSB-first radix select, 8 bits per round, finds each problem's K-th value:
// every CTA histograms its own keys in shared memory, one cluster barrier publishes the
// histograms, and every CTA sums its peers' bins through distributed shared memory and walks
// them - redundantly, so no broadcast is needed.  Two bit masks per thread follow the rounds:
// "live" (equal to the K-th value on all digits so far) and "sel" (already known to rank above it).
// Keys equal to the K-th value are taken in position order (prefix counts by ballot, warp, CTA and
// cluster rank), then a second prefix count over the combined mask places the kept positions.
// The result equals the first K entries of a stable descending sort, exactly.
#pragma once

#include "csp_device.cuh"
#include "csp_internal.cuh"

namespace csp {
namespace sel {
using namespace dev;

constexpr uint32_t kFull = 0xffffffffu;
constexpr int kTeamBarrier = 1;                          // named barrier of a selection team inside a larger CTA

template <int kCsWarps>
struct SelectSmem {
    __align__(16) uint32_t hist[2][4][256];              // ping-pong: a round never zeroes what peers still read
    uint32_t chosen[4];                                  // digit of the K-th value decided in the last round
    int32_t krem[4];                                     // how many are still to be taken among the live keys
    int32_t act[4];
    uint32_t eqcnt[4];                                   // keys equal to the final K-th value
    uint32_t wtie[kCsWarps][4];
    uint32_t wkeep[kCsWarps];
    __align__(16) uint32_t ctie[4];                      // this CTA's totals, read by its peers
    uint32_t ckeep;
};

// barrier over the whole cluster; a cluster of one CTA only needs the CTA barrier
__device__ __forceinline__ void cluster_sync_all(uint32_t csize) {
    if (csize == 1) { __syncthreads(); return; }
    cluster_arrive();
    cluster_wait();
}
__device__ __forceinline__ uint4 ld_shared_u4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}

// kTeam = false: the calling CTA (all kCsThreads threads of it) is one of the cluster that owns unit u.
// kTeam = true: the first kCsThreads threads of a larger CTA own unit u alone (no cluster); they synchronise
// on a named barrier, and the caller puts such a barrier between two units because `sm` is reused.  In this mode the team
// also writes the labels of the kept positions (label side of Eq. 4) to labels_out [B, H_kv, out_capacity] when that is
// not null: it holds every key's label in registers anyway.
template <int kCsThreads, int E, bool kTeam>
__device__ __forceinline__ void select_unit(const SelectArgs& a, const int unit, SelectSmem<kCsThreads / 32>& sm,
                                            uint8_t* const labels_out = nullptr) {
    const int u = kTeam ? unit : int(blockIdx.y);       // the stand-alone kernel's grid row (a special register, not a live value)
    constexpr int kCsWarps = kCsThreads / 32;
    uint32_t (&hist)[2][4][256] = sm.hist;
    uint32_t (&chosen)[4] = sm.chosen;
    int32_t (&krem)[4] = sm.krem;
    int32_t (&act)[4] = sm.act;
    uint32_t (&eqcnt)[4] = sm.eqcnt;
    uint32_t (&wtie)[kCsWarps][4] = sm.wtie;
    uint32_t (&wkeep)[kCsWarps] = sm.wkeep;
    uint32_t (&ctie)[4] = sm.ctie;
    uint32_t& ckeep = sm.ckeep;
    auto sync_cta = [] {
        if constexpr (kTeam) asm volatile("bar.sync %0, %1;" ::"n"(kTeamBarrier), "n"(kCsThreads) : "memory");
        else __syncthreads();
    };
    auto rd_u4 = [](uint32_t addr, uint32_t r) { if constexpr (kTeam) return ld_shared_u4(addr); else return ld_remote_u4(addr, r); };
    auto rd_u32 = [](uint32_t addr, uint32_t r) { if constexpr (kTeam) return ld_shared_u32(addr); else return ld_remote_u32(addr, r); };

    const int b = u / a.n_kv_heads, h = u % a.n_kv_heads;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = kTeam ? 0u : cluster_rank(), csize = kTeam ? 1u : cluster_size();
    auto sync_all = [&] { if constexpr (kTeam) sync_cta(); else cluster_sync_all(csize); };
    const int L = a.seq_lens[b];
    int32_t* const idx = a.keep_idx + int64_t(u) * a.out_capacity;

    // ---- cases decided per unit; the whole cluster leaves together, before any cluster barrier
    if (L < 0 || L > a.max_len) {
        if (tid == 0 && rank == 0) { a.n_out[u] = -1; atomicOr(a.status, CSP_DEV_BAD_LEN); }
        return;
    }
    // Algorithm 1: a cache below its budget T (or too short for a window / recent block) is kept whole
    if (L < a.window || L < a.recent || (a.total_budget && L < a.total_budget[b])) {
        if (L > a.out_capacity) {
            if (tid == 0 && rank == 0) { a.n_out[u] = -1; atomicOr(a.status, CSP_DEV_CAPACITY); }
            return;
        }
        for (int t = int(rank) * kCsThreads + tid; t < L; t += int(csize) * kCsThreads) idx[t] = t;
        if constexpr (kTeam) {
            if (labels_out) {
                const uint8_t* const mod_u = a.modality + int64_t(b) * a.mod_sb + int64_t(h) * a.mod_sh;
                for (int t = tid; t < L; t += kCsThreads) labels_out[int64_t(u) * a.out_capacity + t] = mod_u[t];
            }
        }
        if (tid == 0 && rank == 0) a.n_out[u] = L;
        return;
    }

    const int N = L - a.recent;
    const float* const ss = a.score_self + int64_t(u) * a.max_len;
    const float* const sc = a.score_cross + int64_t(u) * a.max_len;
    const uint8_t* const mod = a.modality + int64_t(b) * a.mod_sb + int64_t(h) * a.mod_sh;
    const int nprob = a.global_mode ? 2 : 4;
    const int32_t* const bud = a.budgets + int64_t(b) * (a.overall ? 1 : nprob);
    const int pc_base = a.global_mode ? 1 : 2;           // first inter-score problem
    const int pc1 = pc_base + 1 < 4 ? pc_base + 1 : 3;

    // ---- keys into registers
    const int warp_base = (int(rank) * kCsWarps + warp) * (32 * E);
    uint32_t ks[E], kc[E];
    uint32_t valid = 0u, vis = 0u;                       // bit e: position in range / visual key
    // team mode: the keys' label bytes, four to a register; with 16 keys per thread the registers are needed
    // elsewhere and the labels of the kept keys are read again at the end
    constexpr bool kKeepLabels = kTeam && E <= 8;
    uint32_t labels[kKeepLabels ? (E + 3) / 4 : 1] = {};
    {
        // all loads are issued before any is used (positions past the end re-read position 0)
        float fs[E], fc[E];
        uint8_t lab[E];
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int t = warp_base + e * 32 + lane;
            const int tc = t < N ? t : 0;
            fs[e] = __ldg(ss + tc);
            fc[e] = __ldg(sc + tc);
            lab[e] = __ldg(mod + tc);
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const bool ok = warp_base + e * 32 + lane < N;
            if (a.overall) fs[e] = fc[e] = fs[e] + fc[e];        // one top-K on the summed score, run twice
            ks[e] = ok ? order_key(fs[e]) : 0u;
            kc[e] = ok ? order_key(fc[e]) : 0u;
            if (ok) valid |= 1u << e;
            if (ok && !a.global_mode && lab[e] != 0) vis |= 1u << e;
            if constexpr (kKeepLabels) labels[e >> 2] |= uint32_t(lab[e]) << (8 * (e & 3));
        }
    }
    if (tid < 4) {
        chosen[tid] = 256u;
        const int32_t k = tid < nprob ? bud[a.overall ? 0 : tid] : 0;
        krem[tid] = k;
        act[tid] = k > 0;
        eqcnt[tid] = 0;
        if (k < 0 && rank == 0) atomicOr(a.status, CSP_DEV_K_CLAMPED);
    }
    sync_cta();

    // Masks over this thread's E keys, per problem kind (_s: intra score, _c: inter score):
    //   live = equal to the K-th value on every digit fixed so far (starts as: competes at all)
    //   sel  = already known to rank above the K-th value
    uint32_t live_s = valid & ((act[0] ? ~vis : 0u) | (act[1] ? vis : 0u));
    uint32_t live_c = valid & ((act[pc_base] ? ~vis : 0u) | (act[pc1] ? vis : 0u));
    uint32_t sel_s = 0u, sel_c = 0u;

    // compare the digit just decided (at bit `at`) with the one chosen for the key's problem
    auto settle = [&](int at) {
        const uint32_t ds0 = chosen[0], ds1 = chosen[1], dc0 = chosen[pc_base], dc1 = chosen[pc1];
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const uint32_t bit = 1u << e;
            const bool v = vis & bit;
            if (live_s & bit) {
                const uint32_t dg = (ks[e] >> at) & 255u, d = v ? ds1 : ds0;
                if (dg > d) sel_s |= bit;
                if (dg != d) live_s &= ~bit;
            }
            if (live_c & bit) {
                const uint32_t dg = (kc[e] >> at) & 255u, d = v ? dc1 : dc0;
                if (dg > d) sel_c |= bit;
                if (dg != d) live_c &= ~bit;
            }
        }
    };

    // ---- radix select, 8 bits per round, most significant first
#pragma unroll 1
    for (int round = 0; round < 4; ++round) {
        const int shift = 24 - 8 * round;
        uint32_t* const hb = &hist[round & 1][0][0];
        for (int i = tid; i < 4 * 256; i += kCsThreads) hb[i] = 0;
        if (round > 0 && (live_s | live_c) != 0u) settle(shift + 8);   // most threads have no live key after a round or two
        sync_cta();
        if (round == 0) {
            // the top byte (sign, high exponent bits) takes very few values: count this thread's keys
            // that share the slot of its first live key and add them with one atomic; twice; then the rest
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                uint32_t slot[E];
                uint32_t todo = which ? live_c : live_s;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const uint32_t v = (vis >> e) & 1u;
                    slot[e] = (which ? uint32_t(pc_base) + v : v) * 256u + ((which ? kc[e] : ks[e]) >> 24);
                }
#pragma unroll
                for (int iter = 0; iter < 2; ++iter) {
                    if (__all_sync(kFull, todo == 0u)) break;           // whole warp done
                    uint32_t first = 0u;
                    bool have = false;
#pragma unroll
                    for (int e = 0; e < E; ++e)
                        if (!have && ((todo >> e) & 1u)) { first = slot[e]; have = true; }
                    uint32_t same = 0u;
#pragma unroll
                    for (int e = 0; e < E; ++e)
                        if (((todo >> e) & 1u) && slot[e] == first) same |= 1u << e;
                    // neighbouring positions mostly share the slot: when the whole warp agrees, one lane adds
                    // the warp's total instead of 32 lanes hitting the same shared-memory word
                    const uint32_t cnt = uint32_t(__popc(same));
                    const uint32_t voters = __ballot_sync(kFull, todo != 0u);
                    const uint32_t f0 = __shfl_sync(kFull, first, voters ? __ffs(voters) - 1 : 0);
                    if (__all_sync(kFull, todo == 0u || first == f0)) {
                        const uint32_t total = __reduce_add_sync(kFull, cnt);
                        if (lane == 0 && total) atomicAdd(&hb[f0], total);
                    } else if (todo != 0u) {
                        atomicAdd(&hb[first], cnt);
                    }
                    todo &= ~same;
                }
                if (todo != 0u) {
#pragma unroll
                    for (int e = 0; e < E; ++e)
                        if ((todo >> e) & 1u) atomicAdd(&hb[slot[e]], 1u);
                }
            }
        } else if ((live_s | live_c) != 0u) {
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const uint32_t v = (vis >> e) & 1u;
                if ((live_s >> e) & 1u) atomicAdd(&hb[v * 256u + ((ks[e] >> shift) & 255u)], 1u);
                if ((live_c >> e) & 1u) atomicAdd(&hb[(uint32_t(pc_base) + v) * 256u + ((kc[e] >> shift) & 255u)], 1u);
            }
        }
        sync_all();                         // every CTA's histogram of this round is complete
        if (warp < nprob && act[warp]) {
            // lane l owns bins 8l..8l+7 of this warp's problem, summed over the cluster
            uint32_t bins[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            const uint32_t local = smem_u32(&hist[round & 1][warp][lane * 8]);
            for (uint32_t r = 0; r < csize; ++r) {
                const uint4 lo = rd_u4(local, r), hi = rd_u4(local + 16, r);
                bins[0] += lo.x; bins[1] += lo.y; bins[2] += lo.z; bins[3] += lo.w;
                bins[4] += hi.x; bins[5] += hi.y; bins[6] += hi.z; bins[7] += hi.w;
            }
            uint32_t ls = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) ls += bins[i];
            uint32_t suf = ls;                           // inclusive suffix sum over lanes
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_down_sync(kFull, suf, d);
                if (lane + d < 32) suf += o;
            }
            int32_t k = krem[warp];
            if (round == 0) {
                const uint32_t total = __shfl_sync(kFull, suf, 0);   // candidates of this problem
                if (uint32_t(k) > total) {
                    k = int32_t(total);
                    if (lane == 0 && rank == 0) atomicOr(a.status, CSP_DEV_K_CLAMPED);
                }
            }
            __syncwarp();
            if (k == 0) {
                if (lane == 0) { act[warp] = 0; krem[warp] = 0; chosen[warp] = 256u; }   // nothing ranks above 256
            } else {
                const uint32_t above = suf - ls;
                if (above < uint32_t(k) && uint32_t(k) <= suf) {
                    uint32_t cum = above;
#pragma unroll
                    for (int i = 7; i >= 0; --i) {
                        if (cum + bins[i] >= uint32_t(k)) {
                            chosen[warp] = uint32_t(lane * 8 + i);
                            krem[warp] = k - int32_t(cum);
                            eqcnt[warp] = bins[i];
                            break;
                        }
                        cum += bins[i];
                    }
                }
            }
        }
        sync_cta();
    }
    if ((live_s | live_c) != 0u) settle(0);
    // live_* now marks the keys equal to their problem's K-th value: krem[p] of the eqcnt[p] such keys
    // are taken, the earliest positions first

    bool any_ties = false;                               // some problem takes only part of its equal keys
#pragma unroll
    for (int p = 0; p < 4; ++p) any_ties |= act[p] != 0 && eqcnt[p] != uint32_t(krem[p]);

    if (!any_ties) {                                     // same decision in every thread of the cluster
        sel_s |= live_s;
        sel_c |= live_c;
    } else {
        // equal-valued keys at earlier positions, per (problem kind, label): s0, s1, c0, c1
        const int32_t take[4] = {krem[0], krem[1], krem[pc_base], krem[pc1]};
        uint32_t tie_base[4];
        tie_base[0] = __reduce_add_sync(kFull, uint32_t(__popc(live_s & ~vis)));
        tie_base[1] = __reduce_add_sync(kFull, uint32_t(__popc(live_s & vis)));
        tie_base[2] = __reduce_add_sync(kFull, uint32_t(__popc(live_c & ~vis)));
        tie_base[3] = __reduce_add_sync(kFull, uint32_t(__popc(live_c & vis)));
        if (lane == 0) {
            wtie[warp][0] = tie_base[0]; wtie[warp][1] = tie_base[1];
            wtie[warp][2] = tie_base[2]; wtie[warp][3] = tie_base[3];
        }
        sync_cta();
        if (tid < 4) {
            uint32_t t = 0;
            for (int w = 0; w < kCsWarps; ++w) t += wtie[w][tid];
            ctie[tid] = t;
        }
        sync_all();
        tie_base[0] = tie_base[1] = tie_base[2] = tie_base[3] = 0;
        for (int r = 0; r < int(rank); ++r) {
            const uint4 t4 = rd_u4(smem_u32(&ctie[0]), r);
            tie_base[0] += t4.x; tie_base[1] += t4.y; tie_base[2] += t4.z; tie_base[3] += t4.w;
        }
        for (int w = 0; w < warp; ++w) {
            tie_base[0] += wtie[w][0]; tie_base[1] += wtie[w][1]; tie_base[2] += wtie[w][2]; tie_base[3] += wtie[w][3];
        }
        const uint32_t lt = (1u << lane) - 1u;
#pragma unroll
        for (int e = 0; e < E; ++e) {                    // position order inside a warp is (e, lane)
            const uint32_t bit = 1u << e;
            const bool v = vis & bit, es = live_s & bit, ec = live_c & bit;
            const uint32_t m0 = __ballot_sync(kFull, es && !v), m1 = __ballot_sync(kFull, es && v);
            const uint32_t m2 = __ballot_sync(kFull, ec && !v), m3 = __ballot_sync(kFull, ec && v);
            if (es && int32_t((v ? tie_base[1] : tie_base[0]) + __popc((v ? m1 : m0) & lt)) < (v ? take[1] : take[0])) sel_s |= bit;
            if (ec && int32_t((v ? tie_base[3] : tie_base[2]) + __popc((v ? m3 : m2) & lt)) < (v ? take[3] : take[2])) sel_c |= bit;
            tie_base[0] += __popc(m0); tie_base[1] += __popc(m1); tie_base[2] += __popc(m2); tie_base[3] += __popc(m3);
        }
    }

    // ---- combined mask (Eq. 3) and its prefix count
    const uint32_t lt_mask = (1u << lane) - 1u;
    const uint32_t keep_bits = a.combine_and ? (sel_s & sel_c) : (sel_s | sel_c);
    const uint32_t n_warp = __reduce_add_sync(kFull, uint32_t(__popc(keep_bits)));
    if (lane == 0) wkeep[warp] = n_warp;
    sync_cta();
    if (tid == 0) {
        uint32_t s = 0;
        for (int w = 0; w < kCsWarps; ++w) s += wkeep[w];
        ckeep = s;
    }
    sync_all();
    uint32_t pos = 0, n_keep = 0;
    for (uint32_t r = 0; r < csize; ++r) {
        const uint32_t v = rd_u32(smem_u32(&ckeep), r);
        n_keep += v;
        if (int(r) < int(rank)) pos += v;
    }
    if (csize > 1) cluster_arrive();                     // no remote read after this point
    for (int w = 0; w < warp; ++w) pos += wkeep[w];

    if (int(n_keep) + a.recent > a.out_capacity) {
        if (tid == 0 && rank == 0) { a.n_out[u] = -1; atomicOr(a.status, CSP_DEV_CAPACITY); }
    } else {
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const bool keep = (keep_bits >> e) & 1u;
            const uint32_t m = __ballot_sync(kFull, keep);
            if (keep) {
                idx[pos + __popc(m & lt_mask)] = warp_base + e * 32 + lane;
                if constexpr (kTeam) {
                    if (labels_out)
                        labels_out[int64_t(u) * a.out_capacity + pos + __popc(m & lt_mask)] =
                            kKeepLabels ? uint8_t(labels[e >> 2] >> (8 * (e & 3))) : mod[warp_base + e * 32 + lane];
                }
            }
            pos += __popc(m);
        }
        if (rank == 0) {
            for (int j = tid; j < a.recent; j += kCsThreads) idx[int(n_keep) + j] = N + j;   // (+) the last R positions
            if constexpr (kTeam) {
                if (labels_out)
                    for (int j = tid; j < a.recent; j += kCsThreads) labels_out[int64_t(u) * a.out_capacity + int(n_keep) + j] = mod[N + j];
            }
            if (tid == 0) a.n_out[u] = int(n_keep) + a.recent;
        }
    }
    if (csize > 1) cluster_wait();                       // peers are done reading this CTA's shared memory
}

}  // namespace sel
}  // namespace csp
