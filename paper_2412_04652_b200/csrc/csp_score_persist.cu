// Persistent variant of the bf16 tcgen05 scoring kernel for many MHA units (window logits Eq. 5,
// n-softmax rows Eq. 7, recent trim, intra/inter query-axis sums Eq. 1).
//
// Used when a launch has more (sequence, head) units than clusters fit on the GPU.  A cluster of C
// CTAs stays resident and walks over units cluster_id, cluster_id + n_clusters, ...  The roles of a
// CTA are decoupled by mbarriers so that the K stream never stops between units:
//   warp 16  TMA producer: runs ahead into the next unit's K tiles as soon as ring stages free up
//   warp 17  MMA issuer: tile i of every unit uses accumulator buffer i of tensor memory (16 buffers of 32
//            columns); it is refilled as soon as pass 2 of the previous unit has read it
//   warp 18  stages Q and the query-label table up to two units ahead (ring of three sets)
//   warps 0-15 two epilogue teams of 8 warps; team j & 1 takes unit j: pass 1 statistics, cluster-wide
//            merge, pass 2 from tensor memory, scores.  While one
//            team waits for its peers' statistics the other one computes.
// While one epilogue team finishes unit j (statistics exchange, pass 2), the producer, the tensor core
// and the other team already work on unit j + 1 in the buffers that pass 2 has released.  The cluster-wide merge of the row statistics
// uses an mbarrier per CTA that all CTAs of the cluster arrive on remotely, so only the epilogue
// warps take part and nobody else is held up.  Every wait is bounded.
//
// Precondition (checked by the launcher): G = 1 and at most 16 tiles per CTA, so that every tile's logits stay
// in tensor memory between the passes.  With a caller-supplied log-sum-exp of the window rows there is no pass 1:
// the epilogue teams go straight to the weights.
#include <mutex>

#include "csp_internal.cuh"
#include "csp_tc.cuh"

namespace csp {
namespace {
using namespace dev;

// barrier over `nthreads` threads (barrier id `id`) that also tells everyone whether any of them saw `pred`
__device__ __forceinline__ bool barrier_any(bool pred, int id, uint32_t nthreads) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "barrier.cta.red.or.pred q, %3, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"(uint32_t(pred)), "r"(nthreads), "r"(id) : "memory");
    return r != 0;
}

constexpr int kTeams = 2;                               // epilogue teams; team p owns tensor-memory half p
constexpr int kTeamWarps = 8;                           // two groups of four warps (one per TMEM lane quarter)
constexpr int kTeamThreads = 32 * kTeamWarps;
constexpr int kEpiWarps = kTeams * kTeamWarps;
constexpr int kPsProducerWarp = kEpiWarps;
constexpr int kPsMmaWarp = kEpiWarps + 1;
constexpr int kPsStageWarp = kEpiWarps + 2;
constexpr int kPsThreads = 32 * (kEpiWarps + 3);        // epilogue warps, producer, MMA issuer, stager
// barrier over the 256 threads of one epilogue team
__device__ __forceinline__ void team_sync(int team) {
    asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "n"(kTeamThreads) : "memory");
}
constexpr int kBufs = 16;                               // tiles whose logits tensor memory holds (32 columns each)
constexpr int kPsMaxStages = 8;
constexpr int kQSets = 3;                               // Q tiles and label tables staged ahead (ring)
constexpr int kMaxCluster = 16;                         // CTAs per cluster (sizes above 8 need the non-portable opt-in)

struct PsSmemPlan {   // byte offsets from the 1024-aligned base
    uint32_t q, wstats, cstats, cvec, dq_mask, dq_val, bars, misc, total;
};
__host__ __device__ inline PsSmemPlan ps_smem_plan(int nh, int stages) {
    PsSmemPlan s;
    uint32_t off = uint32_t(stages) * uint32_t(nh) * kBlockBytes;
    s.q = off;        off += uint32_t(kQSets) * uint32_t(nh) * 32u * 128u;   // staged ahead of the tensor core
    s.wstats = off;   off += 16u * 32u * 8u;                     // [team][warp][column]
    s.cstats = off;   off += 4u * uint32_t(kMaxCluster) * 32u * 8u;   // [unit & 3][rank][row], written by the peers
    s.cvec = off;     off += 2u * 32u * 4u;                      // per team
    s.dq_mask = off;  off += uint32_t(kQSets) * 32u * 4u;
    s.dq_val = off;   off += uint32_t(kQSets) * 32u * 4u;
    s.bars = off;     off += (2u * kPsMaxStages + 3u * kBufs + 3u * kQSets + 2u) * 8u;
    s.misc = off;     off += 32u;     // tmem base, abort flag, n distinct query labels [kQSets]
    s.total = off;
    return s;
}

template <int NH>
__global__ void __launch_bounds__(kPsThreads, 1)
score_tc_persist_kernel(const __grid_constant__ CUtensorMap tmap, const ScoreArgs a, const int n_stages,
                        const int n_units, const int n_clusters) {
    constexpr int KS = NH * 4;
    constexpr int NC = 32;
    constexpr uint32_t kStageBytes = NH * kBlockBytes;
    constexpr uint32_t kQBytes = NH * 32 * 128;
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(NC >> 3) << 17) | (uint32_t(128 >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const PsSmemPlan sp = ps_smem_plan(NH, n_stages);
    float2* const wstats = reinterpret_cast<float2*>(base_ptr + sp.wstats);
    float2* const cstats = reinterpret_cast<float2*>(base_ptr + sp.cstats);
    float* const cvec = reinterpret_cast<float*>(base_ptr + sp.cvec);
    uint32_t* const dq_mask = reinterpret_cast<uint32_t*>(base_ptr + sp.dq_mask);
    uint32_t* const dq_val = reinterpret_cast<uint32_t*>(base_ptr + sp.dq_val);
    const uint32_t full_k = base + sp.bars;
    const uint32_t empty_k = full_k + 8 * kPsMaxStages;
    // logits of tile i ready, one barrier set per epilogue team (= unit parity): a team only ever waits
    // on its own set, one phase per unit it handles, so a parity bit identifies the phase
    const uint32_t tmem_full = empty_k + 8 * kPsMaxStages;        // [2][16]
    const uint32_t tmem_empty = tmem_full + 8 * 2 * kBufs;        // [16] pass 2 done with the tile's logits
    const uint32_t unit_done = tmem_empty + 8 * kBufs;    // [kQSets] epilogue team done with the unit's label table
    const uint32_t q_ready = unit_done + 8 * kQSets;              // [kQSets] Q and label table staged
    const uint32_t q_free = q_ready + 8 * kQSets;                 // [kQSets] tensor core done reading Q
    const uint32_t stats_ready = q_free + 8 * kQSets;             // [2] every CTA of the cluster published its statistics
    volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + sp.misc);
    volatile int* const abort_flag = reinterpret_cast<volatile int*>(base_ptr + sp.misc + 4);
    volatile int* const n_dq = reinterpret_cast<volatile int*>(base_ptr + sp.misc + 8);   // [2]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_rank(), csize = cluster_size();
    const int cid = int(blockIdx.x / csize);
    const int W = a.window;

    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < n_stages; ++s) { mbar_init(full_k + 8 * s, 1); mbar_init(empty_k + 8 * s, 1); }
        for (int i = 0; i < kBufs; ++i) {
            mbar_init(tmem_full + 8 * i, 1);
            mbar_init(tmem_full + 8 * (kBufs + i), 1);
            mbar_init(tmem_empty + 8 * i, 4);
        }
        for (int q = 0; q < kQSets; ++q) {
            mbar_init(unit_done + 8 * q, kTeamWarps);
            mbar_init(q_ready + 8 * q, 1);
            mbar_init(q_free + 8 * q, 1);
        }
        for (int p = 0; p < 2; ++p) mbar_init(stats_ready + 8 * p, csize);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kPsMmaWarp) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512u);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    // peers arrive on this CTA's barriers: nobody may start before every CTA has initialised them
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // what every role needs to know about unit u
    struct Unit { int b, h, L, N, my_all, my_cand; bool skip; };
    auto unit_of = [&](int u) {
        Unit x;
        x.b = u / a.n_kv_heads; x.h = u % a.n_kv_heads;
        if (a.order) {
            // the order list lives in the caller's workspace: an entry that is not a sequence number (the caller
            // overwrote the workspace during the call) must not become an address
            const int ob = a.order[x.b];
            if (ob >= 0 && ob < n_units / a.n_kv_heads) x.b = ob;
            else atomicOr(a.status, CSP_DEV_BAD_LEN);
        }
        int L = a.seq_lens[x.b];
        const bool bad = L < 0 || L > a.max_len;
        x.skip = bad || L < a.window || L < a.recent;
        if (x.skip) L = 0;
        x.L = L;
        x.N = x.skip ? 0 : L - a.recent;
        const int tiles_all = (L + kTileKeys - 1) / kTileKeys, tiles_cand = (x.N + kTileKeys - 1) / kTileKeys;
        x.my_all = tiles_all > int(rank) ? (tiles_all - int(rank) + int(csize) - 1) / int(csize) : 0;
        x.my_cand = tiles_cand > int(rank) ? (tiles_cand - int(rank) + int(csize) - 1) / int(csize) : 0;
        if (x.my_all > kBufs) x.my_all = kBufs;          // never happens (launcher); keeps indices in range
        if (x.my_cand > x.my_all) x.my_cand = x.my_all;
        return x;
    };

    // The j-th unit of this cluster, or -1 when it has none left.  Units are dealt to the clusters in
    // rounds of n_clusters; with the sequences sorted by length the direction alternates from round to
    // round, so that every cluster gets a similar share of long and short ones.  Only the last round can
    // be short: a cluster's list never has a hole.
    auto unit_at = [&](int j) {
        const int pos = (a.order && (j & 1)) ? n_clusters - 1 - cid : cid;
        const int u = j * n_clusters + pos;
        return u < n_units ? u : -1;
    };

    if (warp == kPsProducerWarp) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
            int it = 0;
            for (int j = 0; !*abort_flag; ++j) {
                const int u = unit_at(j);
                if (u < 0) break;
                const Unit x = unit_of(u);
                int row = 0, outer = x.b;          // where the next tile lies (a paged cache looks it up one tile ahead)
                if (x.my_all > 0) tile_coords(a, int(rank), x.b, row, outer);
                for (int i = 0; i < x.my_all; ++i, ++it) {
                    const int slot = it % n_stages;
                    const int row_now = row, outer_now = outer;
                    if (i + 1 < x.my_all) tile_coords(a, (i + 1) * int(csize) + int(rank), x.b, row, outer);
                    mbar_wait(empty_k + 8 * slot, (uint32_t(it / n_stages) & 1u) ^ 1u, abort_flag);
                    if (*abort_flag) break;
                    mbar_expect_tx(full_k + 8 * slot, kStageBytes);
#pragma unroll
                    for (int hb = 0; hb < NH; ++hb)
                        tma_load_4d(base + slot * kStageBytes + hb * kBlockBytes, &tmap, full_k + 8 * slot,
                                    hb * 64, row_now, x.h, outer_now);
                }
            }
            if (*abort_flag) {
                // let copies that were issued land before the CTA's shared memory is given up
                for (int s = 0; s < n_stages; ++s) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(full_k + 8 * s, 0) && !mbar_try_wait(full_k + 8 * s, 1) &&
                           global_ns() - t0 < kWaitLimitNs / 8) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == kPsMmaWarp) {
        // =============================== MMA issuer ===============================
        if (lane == 0) {
            int it = 0;
            for (int j = 0; !*abort_flag; ++j) {
                const int u = unit_at(j);
                if (u < 0) break;
                const Unit x = unit_of(u);
                const uint32_t bph = uint32_t(j) & 1u;                  // every buffer is released once per unit
                const uint32_t my_full = tmem_full + 8 * kBufs * (j & 1);   // barrier set of the team that takes unit j
                const int qs = j % kQSets;
                const uint32_t qph = uint32_t(j / kQSets) & 1u;
                mbar_wait(q_ready + 8 * qs, qph, abort_flag);           // Q of this unit is in shared memory
                const uint32_t q_s = base + sp.q + uint32_t(qs) * kQBytes;
                for (int i = 0; i < x.my_all; ++i, ++it) {
                    const int slot = it % n_stages;
                    mbar_wait(full_k + 8 * slot, uint32_t(it / n_stages) & 1u, abort_flag);
                    // the tile that used this buffer two units back has been through pass 2
                    mbar_wait(tmem_empty + 8 * i, bph ^ 1u, abort_flag);
                    if (*abort_flag) break;
                    tc_fence_after();
                    const uint32_t stage_addr = base + slot * kStageBytes;
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const uint64_t ad = sw128_desc(stage_addr + uint32_t(ks >> 2) * kBlockBytes + uint32_t(ks & 3) * 32u);
                        const uint64_t bd = sw128_desc(q_s + uint32_t(ks >> 2) * (NC * 128u) + uint32_t(ks & 3) * 32u);
                        tc_mma_bf16(tmem_base + uint32_t(i * NC), ad, bd, kIdesc, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(empty_k + 8 * slot);
                    tc_commit(my_full + 8 * i);
                }
                // buffers this unit does not use still flip once per unit: one parity rule for all of them
                for (int i = x.my_all; i < kBufs; ++i) {
                    mbar_wait(tmem_empty + 8 * i, bph ^ 1u, abort_flag);
                    mbar_arrive(my_full + 8 * i);
                }
                tc_commit(q_free + 8 * qs);
            }
        }
        __syncwarp();
    } else if (warp == kPsStageWarp) {
        // =============================== Q / label-table stager ===============================
        for (int j = 0;; ++j) {
            if (__any_sync(0xffffffffu, *abort_flag != 0)) break;        // the whole warp leaves together
            const int u = unit_at(j);
            if (u < 0) break;
            const Unit x = unit_of(u);
            const int qs = j % kQSets;
            const uint32_t qph = uint32_t(j / kQSets) & 1u;
            mbar_wait(q_free + 8 * qs, qph ^ 1u, abort_flag);            // tensor core done with the unit 3 back
            mbar_wait(unit_done + 8 * qs, qph ^ 1u, abort_flag);         // and its epilogue with the label table
            uint8_t* const q_dst = base_ptr + sp.q + qs * kQBytes;
            const uint8_t* qb = static_cast<const uint8_t*>(a.q);
            // lane w stages window row w: all its 16-byte chunks are loaded before any is stored, so the
            // global-memory latency is paid once per unit, not once per chunk
            constexpr int kChunksPerRow = NH * 8;
            {
                const int w = lane;
                uint4 v[kChunksPerRow];
                const bool have = w < W && !x.skip;
                const int64_t e = int64_t(x.b) * a.q_sb + int64_t(x.h) * a.q_sh + int64_t(w) * a.q_st;
                const uint4* src = reinterpret_cast<const uint4*>(qb + e * 2);
#pragma unroll
                for (int c = 0; c < kChunksPerRow; ++c) v[c] = have ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int c = 0; c < kChunksPerRow; ++c) {
                    const uint32_t off = uint32_t(c >> 3) * (NC * 128) + uint32_t(w) * 128 + (uint32_t((c & 7) ^ (w & 7)) << 4);
                    *reinterpret_cast<uint4*>(q_dst + off) = v[c];
                }
            }
            // table of the distinct labels of the window queries and the columns carrying each
            const uint8_t* modp = a.modality + int64_t(x.b) * a.mod_sb + int64_t(x.h) * a.mod_sh;
            const uint32_t ql = (lane < W && !x.skip) ? modp[x.L - W + lane] : 0xFFFFFFFFu;
            int count = 0;
            for (int jq = 0; jq < W; ++jq) {
                const uint32_t vj = __shfl_sync(0xffffffffu, ql, jq);
                const uint32_t same = __ballot_sync(0xffffffffu, ql == vj);
                if ((same & ((1u << jq) - 1u)) == 0u) {               // no earlier column has this label
                    if (lane == 0) { dq_val[qs * 32 + count] = vj; dq_mask[qs * 32 + count] = same; }
                    ++count;
                }
            }
            if (lane == 0) n_dq[qs] = x.skip ? 0 : count;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make Q visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(q_ready + 8 * qs);
        }
    } else {
        // =============================== epilogue warps ===============================
        const int team = warp / kTeamWarps, tw = warp % kTeamWarps;   // team-local warp index
        const int quarter = tw & 3, group = tw >> 2;
        const int lq = lane & 3, lr = lane >> 2;
        const float scale2 = a.scale_log2;
        const uint32_t wmask = W >= 32 ? 0xFFFFFFFFu : ((1u << W) - 1u);
        float2* const wst = wstats + team * (kTeamWarps * 32);
        float* const cv_team = cvec + team * 32;
        for (int j = team;; j += kTeams) {
            const int u = unit_at(j);
            if (u < 0) break;
            if (barrier_any(*abort_flag != 0, 1 + team, kTeamThreads)) break;   // the whole team leaves together
            const Unit x = unit_of(u);
            const int p = j & 1;
            const uint32_t ph = uint32_t(j >> 1) & 1u;
            const uint32_t my_full = tmem_full + 8 * kBufs * team;   // this team's barrier set; one phase per unit it takes
            const int first_masked_key = x.L - W;
            const uint8_t* modp = a.modality + int64_t(x.b) * a.mod_sb + int64_t(x.h) * a.mod_sh;
            if (tw == 0 && lane == 0 && rank == 0) {
                const int Lraw = a.seq_lens[x.b];
                if (Lraw < 0 || Lraw > a.max_len) atomicOr(a.status, CSP_DEV_BAD_LEN);
            }

            const int qs = j % kQSets;
            // With the rows' log-sum-exp supplied by the caller there is no pass 1 and nothing to exchange: the
            // additive constants follow from it directly and pass 2 consumes the tiles as they arrive.
            if (a.lse) {
                if (tw == 0) {
                    const float m = (lane < W && !x.skip)
                                        ? a.lse[(int64_t(x.b) * a.n_kv_heads + x.h) * W + lane] * 1.4426950408889634f : 0.f;
                    const float denom = a.n * ex2f(-m) + 1.f;          // (max, sum) = (lse, 1)
                    cv_team[lane] = lane < W ? lg2f(a.weight / denom) - m : -INFINITY;
                    mbar_wait(q_ready + 8 * qs, uint32_t(j / kQSets) & 1u, abort_flag);   // label table of this unit
                }
            } else {
            // ---------------------------------- pass 1 ----------------------------------
            float m_run[8], z_run[8];
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) { m_run[jj] = kNeg; z_run[jj] = 0.f; }
            for (int i = group; i < x.my_all; i += 2) {
                const int buf = i;
                const int tile = i * int(csize) + int(rank);
                mbar_wait(my_full + 8 * buf, ph, abort_flag);
                tc_fence_after();
                const bool masked = (tile + 1) * kTileKeys > first_masked_key;
                const int t_base = tile * kTileKeys + quarter * 32 + lr;
                uint32_t v0[16], v1[16];
                tc_ld_16x32(v0, tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(buf * NC));
                tc_ld_16x32(v1, tmem_base + (uint32_t(quarter * 32 + 16) << 16) + uint32_t(buf * NC));
                tc_wait_ld();
                if (!masked) stats_block<4>(v0, v1, m_run, z_run, scale2);
                else stats_block_masked<4>(v0, v1, m_run, z_run, scale2, t_base, first_masked_key, W, lq * 2);
            }
            // merge: lanes holding the same columns, then warps, then the CTAs of the cluster
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
#pragma unroll
                for (int d = 4; d <= 16; d <<= 1) {
                    const float om = __shfl_xor_sync(0xffffffffu, m_run[jj], d);
                    const float oz = __shfl_xor_sync(0xffffffffu, z_run[jj], d);
                    merge_stats(m_run[jj], z_run[jj], om, oz);
                }
                if (lr == 0) wst[tw * 32 + (jj >> 1) * 8 + lq * 2 + (jj & 1)] = make_float2(m_run[jj], z_run[jj]);
            }
            team_sync(team);
            if (tw == 0) {
                // lane l owns window row l: merge the team's warps, push the result into every peer's
                // shared memory (slot [p][my rank][l]) and tell the peer; then wait for all peers' pushes
                float2 v[kTeamWarps];
#pragma unroll
                for (int w = 0; w < kTeamWarps; ++w) v[w] = wst[w * 32 + lane];
#pragma unroll
                for (int d = 1; d < kTeamWarps; d <<= 1)                  // pairwise tree, fixed order
#pragma unroll
                    for (int w = 0; w < kTeamWarps; w += 2 * d) merge_stats(v[w].x, v[w].y, v[w + d].x, v[w + d].y);
                const int slot4 = j & 3;   // a peer can only overwrite a slot four units later, after this CTA's arrive for j + 2
                const uint32_t mine = smem_u32(&cstats[(slot4 * kMaxCluster + int(rank)) * 32 + lane]);
                for (uint32_t r = 0; r < csize; ++r) st_remote_f2(mine, r, v[0]);
                asm volatile("fence.acq_rel.cluster;" ::: "memory");
                __syncwarp();
                if (lane < int(csize)) mbar_arrive_remote(stats_ready + 8 * p, uint32_t(lane));
                mbar_wait_cluster(stats_ready + 8 * p, ph, abort_flag);
                // merged in rank order (fixed, so results are reproducible); this sits on the unit's critical path, so no
                // work is spent on ranks the cluster does not have (a tree over all sixteen possible ranks, guarded per
                // node, measured 8 % slower on the whole kernel)
                float m = kNeg, z = 0.f;
                for (int r = 0; r < int(csize); ++r) {
                    const float2 cr = cstats[(slot4 * kMaxCluster + r) * 32 + lane];
                    merge_stats(m, z, cr.x, cr.y);
                }
                // weight of 2^(x - m) is 1 / (n 2^-m + Z); fold it and -m into one additive constant
                const float denom = a.n * ex2f(-m) + z;
                cv_team[lane] = lane < W ? lg2f(a.weight / denom) - m : -INFINITY;
                mbar_wait(q_ready + 8 * qs, uint32_t(j / kQSets) & 1u, abort_flag);   // label table of this unit
            }
            }   // pass 1 and the exchange of its statistics
            team_sync(team);

            // ---------------------------------- pass 2 ----------------------------------
            float* const out_s = a.score_self + (int64_t(x.b) * a.n_kv_heads + x.h) * a.max_len;
            float* const out_c = a.score_cross + (int64_t(x.b) * a.n_kv_heads + x.h) * a.max_len;
            const int ndq = n_dq[qs];
            auto t_of = [&](int i) { return (i * int(csize) + int(rank)) * kTileKeys + quarter * 32 + lane; };
            uint32_t kmod_next = (group < x.my_cand && t_of(group) < x.N) ? modp[t_of(group)] : 0u;
            for (int i = group; i < kBufs; i += 2) {
                const int buf = i;
                // without a pass 1 nobody has waited for this unit's logits yet
                if (a.lse && i < x.my_all) { mbar_wait(my_full + 8 * buf, ph, abort_flag); tc_fence_after(); }
                if (i >= x.my_cand) {                                    // nothing to score: just hand the buffer back
                    if (i >= x.my_all) mbar_wait(my_full + 8 * buf, ph, abort_flag);     // keep phases in step
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tmem_empty + 8 * buf);
                    continue;
                }
                const int t = t_of(i);
                const uint32_t kmod = kmod_next;
                kmod_next = (i + 2 < x.my_cand && t_of(i + 2) < x.N) ? modp[t_of(i + 2)] : 0u;
                uint32_t same = 0u;                                        // window columns with the key's label
                for (int q = 0; q < ndq; ++q) same = dq_val[qs * 32 + q] == kmod ? dq_mask[qs * 32 + q] : same;
                const int delta = t - first_masked_key;                    // column w sees the key iff w >= delta
                const uint32_t vis = delta <= 0 ? wmask : (delta >= 32 ? 0u : (wmask & (0xFFFFFFFFu << delta)));
                const uint32_t add_s = same & vis, add_c = ~same & vis;
                float s0 = 0.f, s1 = 0.f, c0 = 0.f, c1 = 0.f;
                float2 p01 = make_float2(0.f, 0.f), p23 = make_float2(0.f, 0.f);   // the plain sums
                const uint32_t row_addr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(buf * NC);
                // The whole row of logits goes to registers first and the buffer is handed back at once: the
                // tensor core refills it (next unit) while the weights are still being computed here.
                uint32_t va[16], vb[16];
                tc_ld_row16(va, row_addr);
                tc_ld_row16(vb, row_addr + 16u);
                tc_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tmem_empty + 8 * buf);          // the tensor core may refill this buffer
                // Common case: every window query carries the same label and no column of this tile is
                // hidden.  Then a key's weights all go to one of the two sums, chosen once per key, and the
                // columns beyond W add exact zeros (their constant is -inf): plain sums, no selection.
                const bool plain = ndq == 1 && (i * int(csize) + int(rank) + 1) * kTileKeys <= first_masked_key;
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t (&cur)[16] = ch ? vb : va;
                    const float4* cv = reinterpret_cast<const float4*>(cv_team + ch * 16);
                    if (plain) {
                        // two-wide fp32 instructions: same roundings and order as four scalar sums
                        const float2 sc2 = make_float2(scale2, scale2);
#pragma unroll
                        for (int j4 = 0; j4 < 4; ++j4) {
                            const float4 cc = cv[j4];
                            p01 = __fadd2_rn(p01, ex2f2(__ffma2_rn(make_float2(__uint_as_float(cur[j4 * 4 + 0]), __uint_as_float(cur[j4 * 4 + 1])),
                                                                   sc2, make_float2(cc.x, cc.y))));
                            p23 = __fadd2_rn(p23, ex2f2(__ffma2_rn(make_float2(__uint_as_float(cur[j4 * 4 + 2]), __uint_as_float(cur[j4 * 4 + 3])),
                                                                   sc2, make_float2(cc.z, cc.w))));
                        }
                        continue;
                    }
                    const uint32_t as = add_s >> (ch * 16), ac = add_c >> (ch * 16);
#pragma unroll
                    for (int j4 = 0; j4 < 4; ++j4) {
                        const float4 cc = cv[j4];
                        const float p0 = ex2f(fmaf(__uint_as_float(cur[j4 * 4 + 0]), scale2, cc.x));
                        const float p1 = ex2f(fmaf(__uint_as_float(cur[j4 * 4 + 1]), scale2, cc.y));
                        const float p2 = ex2f(fmaf(__uint_as_float(cur[j4 * 4 + 2]), scale2, cc.z));
                        const float p3 = ex2f(fmaf(__uint_as_float(cur[j4 * 4 + 3]), scale2, cc.w));
                        s0 += (as >> (j4 * 4 + 0)) & 1u ? p0 : 0.f; c0 += (ac >> (j4 * 4 + 0)) & 1u ? p0 : 0.f;
                        s1 += (as >> (j4 * 4 + 1)) & 1u ? p1 : 0.f; c1 += (ac >> (j4 * 4 + 1)) & 1u ? p1 : 0.f;
                        s0 += (as >> (j4 * 4 + 2)) & 1u ? p2 : 0.f; c0 += (ac >> (j4 * 4 + 2)) & 1u ? p2 : 0.f;
                        s1 += (as >> (j4 * 4 + 3)) & 1u ? p3 : 0.f; c1 += (ac >> (j4 * 4 + 3)) & 1u ? p3 : 0.f;
                    }
                }
                if (plain) {
                    const float total = (p01.x + p01.y) + (p23.x + p23.y);
                    s0 = same ? total : 0.f; s1 = 0.f;
                    c0 = same ? 0.f : total; c1 = 0.f;
                }
                if (t < x.N) { out_s[t] = s0 + s1; out_c[t] = c0 + c1; }
            }
            // the label table and Q of this parity may now be restaged
            __syncwarp();
            if (lane == 0) mbar_arrive(unit_done + 8 * qs);
        }
        if (*abort_flag && tw == 0 && lane == 0) atomicOr(a.status, CSP_DEV_TIMEOUT);
    }

    // every warp: give tensor memory back, then keep shared memory alive until the peers are done
    tc_fence_before();
    __syncthreads();
    if (warp == kPsMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512u);
    }
    cluster_arrive();
    cluster_wait();
}

template <int NH>
csp_status launch_nh(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, int c_min, cudaStream_t s,
                     bool* taken) {
    const int units = p.batch * p.n_kv_heads;
    const int fixed = int(ps_smem_plan(NH, 0).total) + 1024;
    int stages = (227 * 1024 - fixed) / (NH * kBlockBytes);
    if (stages > 6) stages = 6;
    if (stages < 2) return CSP_OK;
    const size_t smem = ps_smem_plan(NH, stages).total + 1024;
    auto kern = score_tc_persist_kernel<NH>;
    static std::atomic<bool> configured[kMaxDevices];
    static std::atomic<bool> wide_ok[kMaxDevices];            // cluster sizes above 8 have been allowed for this kernel
    static std::atomic<int> resident[kMaxDevices][kMaxCluster + 1];   // clusters of each size that fit on the device at once
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return CSP_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return CSP_OK;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kPsThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (!raise_smem_limit(kern, 227 * 1024, configured)) return CSP_ERR_CUDA;
    // Sizes above 8 need the kernel's non-portable opt-in.  It is switched on only around a query or a launch that
    // needs it (launches of the portable sizes ran 3 % slower with it left on), under a lock because it is a
    // property of the kernel, not of the launch.
    static std::mutex wide_mutex;
    auto set_wide = [&](bool on) {
        if (wide_ok[dev].load(std::memory_order_relaxed) == on) return;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, on ? 1 : 0) != cudaSuccess) cudaGetLastError();
        wide_ok[dev].store(on, std::memory_order_relaxed);
    };
    std::lock_guard<std::mutex> lock(wide_mutex);
    const int sms = sm_count();
    auto clusters_of = [&](int c) {
        int n = resident[dev][c].load(std::memory_order_relaxed);
        if (n == 0) {
            set_wide(c > 8);
            attr[0].val.clusterDim.x = c;
            cfg.gridDim = dim3((sms / c) * c, 1, 1);
            int q = 0;
            if (cudaOccupancyMaxActiveClusters(&q, kern, &cfg) != cudaSuccess || q <= 0) { cudaGetLastError(); q = -1; }
            n = q;
            resident[dev][c].store(n, std::memory_order_relaxed);
        }
        return n > 0 ? n : 0;
    };
    // Cluster size: the smallest that keeps a unit's logits in tensor memory, unless a larger one covers at least 5 % more
    // SMs (clusters must sit inside one GPC: on a B200 sizes 4 and 8 cover 132 and 120 of the 148 SMs, size 9 covers 135).
    int c = c_min, covered = clusters_of(c_min) * c_min;
    for (int cc = c_min + 1; cc <= kMaxCluster; ++cc) {
        const int cov = clusters_of(cc) * cc;
        if (cov * 100 >= covered * 105) { c = cc; covered = cov; }
    }
    const int n_clusters = clusters_of(c);
    if (n_clusters <= 0) return CSP_OK;
    if (units < 2 * n_clusters) return CSP_OK;           // too few units for a resident loop to pay off
    attr[0].val.clusterDim.x = c;
    cfg.gridDim = dim3(n_clusters * c, 1, 1);
    set_wide(c > 8);
    if (cudaLaunchKernelEx(&cfg, kern, tmap, a, stages, units, n_clusters) != cudaSuccess) {
        cudaGetLastError();
        return CSP_ERR_CUDA;
    }
    *taken = true;
    return CSP_OK;
}

}  // namespace

// Launches the persistent kernel if the shape qualifies; *taken tells whether it did.
csp_status launch_score_persist(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s,
                                bool* taken) {
    *taken = false;
    if (a.group != 1 || a.hist != nullptr) return CSP_OK;
    const int row_bytes = p.head_dim * 2;
    if (row_bytes != 128 && row_bytes != 256) return CSP_OK;
    const int max_tiles = (p.max_len + kTileKeys - 1) / kTileKeys;
    const int c = (max_tiles + kBufs - 1) / kBufs > 0 ? (max_tiles + kBufs - 1) / kBufs : 1;   // smallest size that keeps the logits
    if (c > kMaxCluster) return CSP_OK;
    return row_bytes == 128 ? launch_nh<1>(p, a, tmap, c, s, taken) : launch_nh<2>(p, a, tmap, c, s, taken);
}

}  // namespace csp
