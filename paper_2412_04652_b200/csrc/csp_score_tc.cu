// Scoring kernel for bf16 caches on the 5th-generation tensor cores (tcgen05 + tensor memory):
// window logits (Eq. 5), n-softmax rows (Eq. 7), recent trim, head-group mean and the intra/inter
// query-axis sums (Eq. 1), for one layer.
//
// One thread-block cluster of C CTAs owns one (sequence, KV head) unit; 128-key tiles of K are
// dealt round-robin to its CTAs.  Inside a CTA
//   warp 8      TMA producer: K tiles -> ring of 128B-swizzled shared-memory stages
//   warp 9      one thread issues tcgen05.mma: D[128 keys x 32G queries] = K_tile . Q^T, fp32
//               accumulators in tensor memory, several tiles in flight (ring of TMEM buffers)
//   warps 0-7   epilogue, two groups of four warps taking alternate tiles, reading TMEM.  For G >= 3
//               a second set of eight warps works on the same tiles: each set takes 16 of the 32
//               window columns of every query head, which halves the per-thread statistics and
//               doubles the warps that hide the latency of tensor-memory loads and exponentials
// The same tile stream runs twice:
//   pass 1  all tiles of the unit: per window row a running (max, sum of 2^(x-max)); merged over
//           lanes, warps and - through distributed shared memory - the CTAs of the cluster
//   pass 2  candidate tiles again - from tensor memory where the logits were kept, else recomputed
//           from K (L2 hits): one thread per key reads its row of logits,
//           weight = 2^(x*scale + c_w) with c_w = log2(1 / (G (n 2^-m + Z))) - m, added to the key's
//           intra or inter sum by label equality; no cross-thread reduction is left, and the two
//           score vectors are written fully coalesced.
// Summation orders are fixed: results are bit-reproducible run to run.
#include "csp_internal.cuh"
#include "csp_tc.cuh"

namespace csp {
namespace {
using namespace dev;

// epilogue organisation for a group of G query heads per KV head
template <int G> struct EpiPlan {
    static constexpr bool kSplit = G >= 3;              // two warp sets, each with half of the window columns
    static constexpr int kSets = kSplit ? 2 : 1;
    static constexpr bool kFmaExp = kSplit;             // one pair of exponentials in eight on the FMA pipe
    static constexpr int kWarps = 8 * kSets;
    static constexpr int kEpiThreads = 32 * kWarps;
    static constexpr int kBlocks = kSplit ? 2 : 4;      // 8-column blocks per head and thread in pass 1
    static constexpr int kCols = 8 * kBlocks;           // window columns of a head that one set handles
    static constexpr int kProducerWarp = kWarps;
    static constexpr int kMmaWarp = kWarps + 1;
    static constexpr int kThreads = 32 * (kWarps + 2);
};
constexpr int kMaxStages = 8;
constexpr int kMaxTmemBufs = 16;

// Tensor memory (512 columns x 128 lanes of fp32 per SM) holds one accumulator of 32G columns per key
// tile.  If all tiles of the CTA fit into its share they simply stay there after pass 1 and pass 2
// reads them back: no second pass over K.  Otherwise all but 2-4 buffers keep the first tiles and the
// rest cycle through the remaining "streaming" buffers in both passes.
// A CTA either owns the SM (512 columns, up to 6 K stages) or shares it with a second CTA (256
// columns, 3 stages, MHA only), so that one CTA's barrier and epilogue phases overlap the other's
// streaming.
template <int G> struct TmemPlan {
    static constexpr int kCols = 32 * G;               // accumulator columns per tile
    static constexpr int kBufs = 512 / kCols;          // buffers when the CTA owns the SM
    static constexpr int kBufsShared = 256 / kCols;    // buffers when two CTAs share the SM
};

struct TcSmemPlan {   // byte offsets from the 1024-aligned base
    uint32_t q, wstats, cstats, cvec, xchg, dq_mask, dq_val, bars, misc, hist, total;
};
constexpr int kHistBins = CSP_HIST_BINS;
__host__ __device__ inline TcSmemPlan tc_smem_plan(int nh, int g, int stages, bool with_hist) {
    TcSmemPlan s;
    uint32_t off = uint32_t(stages) * uint32_t(nh) * kBlockBytes;
    s.q = off;        off += uint32_t(nh) * uint32_t(g) * 32u * 128u;
    s.wstats = off;   off += 8u * uint32_t(g) * 32u * 8u;   // [warp][head][column of its set]
    s.cstats = off;   off += uint32_t(g) * 32u * 8u;
    s.cvec = off;     off += uint32_t(g) * 32u * 4u;
    s.xchg = off;     off += 2u * 2u * 128u * 8u;       // [parity][group][key row]: set 1's partial sums
    s.dq_mask = off;  off += 32u * 4u;
    s.dq_val = off;   off += 32u * 4u;
    s.bars = off;     off += (2u * kMaxStages + 2u * kMaxTmemBufs + 1u) * 8u;
    s.misc = off;     off += 16u;                       // tmem base, abort flag, n distinct query labels
    s.hist = off;     off += with_hist ? 16u * 2u * uint32_t(kHistBins) * 4u : 0u;   // [epilogue warp][intra, inter][bin]
    s.total = off;
    return s;
}

// kHist: the distribution diagnostic (csp_weight_histogram) rides on pass 2; a separate instantiation, so that
// the scoring kernels proper carry none of its code
template <int NH, int G, bool kHist>
__global__ void __launch_bounds__(EpiPlan<G>::kThreads, (G == 1 && NH <= 2) ? 2 : 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmap, const ScoreArgs a, const int n_stages,
                const int tmem_cols) {
    using EP = EpiPlan<G>;
    constexpr int kProducerWarp = EP::kProducerWarp, kMmaWarp = EP::kMmaWarp;
    constexpr int KS = NH * 4;                          // MMAs (K = 16 elements = 32 bytes) per tile
    constexpr int NC = TmemPlan<G>::kCols;
    const int TB = tmem_cols / NC;                      // accumulator buffers this CTA owns
    const int NS = TB >= 8 ? 4 : 2;                     // of which streaming buffers when not all tiles fit
    constexpr uint32_t kStageBytes = NH * kBlockBytes;
    // instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major, M = 128, N = NC
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(NC >> 3) << 17) | (uint32_t(128 >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    constexpr bool want_hist = kHist;
    const TcSmemPlan sp = tc_smem_plan(NH, G, n_stages, want_hist);
    const uint32_t q_s = base + sp.q;
    float2* const wstats = reinterpret_cast<float2*>(base_ptr + sp.wstats);
    float2* const cstats = reinterpret_cast<float2*>(base_ptr + sp.cstats);
    float* const cvec = reinterpret_cast<float*>(base_ptr + sp.cvec);
    float2* const xchg = reinterpret_cast<float2*>(base_ptr + sp.xchg);
    uint32_t* const dq_mask = reinterpret_cast<uint32_t*>(base_ptr + sp.dq_mask);
    uint32_t* const dq_val = reinterpret_cast<uint32_t*>(base_ptr + sp.dq_val);
    const uint32_t full_k = base + sp.bars;
    const uint32_t empty_k = full_k + 8 * kMaxStages;
    const uint32_t tmem_full = empty_k + 8 * kMaxStages;
    const uint32_t tmem_empty = tmem_full + 8 * kMaxTmemBufs;
    const uint32_t q_ready = tmem_empty + 8 * kMaxTmemBufs;
    volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + sp.misc);
    volatile int* const abort_flag = reinterpret_cast<volatile int*>(base_ptr + sp.misc + 4);
    volatile int* const n_dq = reinterpret_cast<volatile int*>(base_ptr + sp.misc + 8);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = blockIdx.y;
    int b = int(blockIdx.z);
    if (a.order) {
        // the order list lives in the caller's workspace: an entry that is not a sequence number must not become an address
        const int ob = a.order[b];
        if (ob >= 0 && ob < int(gridDim.z)) b = ob;
        else if (threadIdx.x == 0) atomicOr(a.status, CSP_DEV_BAD_LEN);
    }
    const uint32_t rank = cluster_rank(), csize = cluster_size();

    int L = a.seq_lens[b];
    const bool bad_len = L < 0 || L > a.max_len;
    const bool skip = bad_len || L < a.window || L < a.recent;
    if (bad_len && tid == 0 && rank == 0) atomicOr(a.status, CSP_DEV_BAD_LEN);
    if (skip) L = 0;
    const int W = a.window;
    const int N = skip ? 0 : L - a.recent;
    const int tiles_all = a.lse ? 0 : (L + kTileKeys - 1) / kTileKeys;
    const int tiles_cand = (N + kTileKeys - 1) / kTileKeys;
    const int my_all = tiles_all > int(rank) ? (tiles_all - int(rank) + int(csize) - 1) / int(csize) : 0;
    const int my_cand = tiles_cand > int(rank) ? (tiles_cand - int(rank) + int(csize) - 1) / int(csize) : 0;
    // tiles [0, kept) of this CTA keep their logits in tensor memory between the passes
    const int kept = my_all <= TB ? my_all : TB - NS;
    const int streamed1 = my_all - kept;                               // streamed tiles of pass 1
    const int streamed2 = my_cand > kept ? my_cand - kept : 0;         // tiles recomputed in pass 2
    const int total = my_all + streamed2;                              // K tiles loaded by this CTA
    // TMEM buffer and mbarrier parity of tile i of pass `second`
    auto buf_of = [&](int i, int second) { return i < kept ? i : kept + ((second ? streamed1 : 0) + i - kept) % NS; };
    auto par_of = [&](int i, int second) {
        return i < kept ? 0u : uint32_t(((second ? streamed1 : 0) + i - kept) / NS) & 1u;
    };

    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < n_stages; ++s) { mbar_init(full_k + 8 * s, 1); mbar_init(empty_k + 8 * s, 1); }
        for (int i = 0; i < TB; ++i) { mbar_init(tmem_full + 8 * i, 1); mbar_init(tmem_empty + 8 * i, 4 * EP::kSets); }
        mbar_init(q_ready, EP::kWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), uint32_t(tmem_cols));
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == kProducerWarp) {
        // =============================== TMA producer ===============================
        cluster_arrive();                         // cluster barrier 1: nothing of ours to publish
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
            auto tile_of = [&](int it) { return (it < my_all ? it : it - my_all + kept) * int(csize) + int(rank); };
            int row = 0, outer = b;                // where the next tile lies (a paged cache looks it up one tile ahead)
            if (total > 0) tile_coords(a, tile_of(0), b, row, outer);
            for (int it = 0; it < total; ++it) {
                const int slot = it % n_stages;
                const uint32_t round = uint32_t(it / n_stages);
                const int row_now = row, outer_now = outer;
                if (it + 1 < total) tile_coords(a, tile_of(it + 1), b, row, outer);
                mbar_wait(empty_k + 8 * slot, (round & 1u) ^ 1u, abort_flag);
                if (*abort_flag) break;
                mbar_expect_tx(full_k + 8 * slot, kStageBytes);
#pragma unroll
                for (int hb = 0; hb < NH; ++hb)
                    tma_load_4d(base + slot * kStageBytes + hb * kBlockBytes, &tmap, full_k + 8 * slot,
                                hb * 64, row_now, h, outer_now);
            }
            if (*abort_flag) {
                // let copies that were issued land before the CTA's shared memory is given up
                const int issued = total < n_stages ? total : n_stages;
                for (int s = 0; s < issued; ++s) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(full_k + 8 * s, 0) && !mbar_try_wait(full_k + 8 * s, 1) &&
                           global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
        __syncwarp();
        cluster_wait();
    } else if (warp == kMmaWarp) {
        // =============================== MMA issuer ===============================
        cluster_arrive();
        if (lane == 0) {
            mbar_wait(q_ready, 0, abort_flag);
            for (int it = 0; it < total; ++it) {
                const int slot = it % n_stages;
                const int second = it >= my_all;
                const int i = second ? it - my_all + kept : it;        // tile index within its pass
                const int buf = buf_of(i, second);
                mbar_wait(full_k + 8 * slot, uint32_t(it / n_stages) & 1u, abort_flag);
                if (i >= kept) mbar_wait(tmem_empty + 8 * buf, par_of(i, second) ^ 1u, abort_flag);
                if (*abort_flag) break;
                tc_fence_after();
                const uint32_t stage_addr = base + slot * kStageBytes;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const uint64_t ad = sw128_desc(stage_addr + uint32_t(ks >> 2) * kBlockBytes + uint32_t(ks & 3) * 32u);
                    const uint64_t bd = sw128_desc(q_s + uint32_t(ks >> 2) * (NC * 128u) + uint32_t(ks & 3) * 32u);
                    tc_mma_bf16(tmem_base + uint32_t(buf * NC), ad, bd, kIdesc, ks > 0 ? 1u : 0u);
                }
                tc_commit(empty_k + 8 * slot);    // stage may be refilled once these MMAs have read it
                tc_commit(tmem_full + 8 * buf);   // accumulator ready for the epilogue
            }
        }
        __syncwarp();
        cluster_wait();
    } else {
        // =============================== epilogue warps ===============================
        const int set = warp >> 3;                          // which half of the window columns
        const int quarter = warp & 3, group = (warp >> 2) & 1;
        const int lq = lane & 3, lr = lane >> 2;
        const int cofs = set * EP::kCols;                   // this warp's columns of every head: [cofs, cofs + kCols)
        auto epi_sync = [] { asm volatile("bar.sync 1, %0;" ::"n"(EP::kEpiThreads) : "memory"); };
        const uint8_t* modp = a.modality + int64_t(b) * a.mod_sb + int64_t(h) * a.mod_sh;

        // stage Q of this KV group: row (g*32 + w), 128-byte column blocks, 16-byte chunks XOR-swizzled
        if (!skip) {
            const uint8_t* qb = static_cast<const uint8_t*>(a.q);
            constexpr int kChunksPerRow = NH * 8;
            for (int i = tid; i < G * 32 * kChunksPerRow; i += EP::kEpiThreads) {
                const int r = i / kChunksPerRow, c = i % kChunksPerRow;
                const int g = r >> 5, w = r & 31;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (w < W) {
                    const int64_t e = int64_t(b) * a.q_sb + int64_t(h * G + g) * a.q_sh + int64_t(w) * a.q_st;
                    v = *reinterpret_cast<const uint4*>(qb + e * 2 + c * 16);
                }
                const uint32_t off = uint32_t(c >> 3) * (NC * 128) + uint32_t(r) * 128 + (uint32_t((c & 7) ^ (r & 7)) << 4);
                *reinterpret_cast<uint4*>(base_ptr + sp.q + off) = v;
            }
        } else {
            for (int i = tid; i < NH * NC * 8; i += EP::kEpiThreads)
                *reinterpret_cast<uint4*>(base_ptr + sp.q + i * 16) = make_uint4(0, 0, 0, 0);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make Q visible to the tensor core
        __syncwarp();
        if (lane == 0) mbar_arrive(q_ready);

        // table of the distinct labels of the window queries and the columns carrying each
        if (warp == 0) {
            const uint32_t ql = (lane < W && !skip) ? modp[L - W + lane] : 0xFFFFFFFFu;
            int count = 0;
            for (int j = 0; j < W; ++j) {
                const uint32_t vj = __shfl_sync(0xffffffffu, ql, j);
                const uint32_t same = __ballot_sync(0xffffffffu, ql == vj);
                const bool first = (same & ((1u << j) - 1u)) == 0u;       // no earlier column has this label
                if (first) {
                    if (lane == 0) { dq_val[count] = vj; dq_mask[count] = same; }
                    ++count;
                }
            }
            if (lane == 0) *n_dq = skip ? 0 : count;
        }

        const float scale2 = a.scale_log2;
        const int first_masked_key = L - W;       // keys beyond this may be hidden from some window row
        // histogram of log2(weight) per query head: the exponent of pass 2 is log2(weight x mean factor)
        uint32_t* const whist = reinterpret_cast<uint32_t*>(base_ptr + sp.hist) + warp * 2 * kHistBins;
        const float hist_shift = want_hist ? -lg2f(a.weight) - CSP_HIST_LO : 0.f;
        if (want_hist)
            for (int j = lane; j < 2 * kHistBins; j += 32) whist[j] = 0u;

        // ---------------------------------- pass 1 ----------------------------------
        constexpr int NB = EP::kBlocks;
        float m_run[G][2 * NB], z_run[G][2 * NB];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int jj = 0; jj < 2 * NB; ++jj) { m_run[g][jj] = kNeg; z_run[g][jj] = 0.f; }

        for (int i = group; i < my_all; i += 2) {
            const int buf = buf_of(i, 0);
            const int tile = i * int(csize) + int(rank);
            mbar_wait(tmem_full + 8 * buf, par_of(i, 0), abort_flag);
            tc_fence_after();
            const bool masked = (tile + 1) * kTileKeys > first_masked_key;
            const int t_base = tile * kTileKeys + quarter * 32 + lr;
#pragma unroll
            for (int g = 0; g < G; ++g) {
                uint32_t v0[4 * NB], v1[4 * NB];
                const uint32_t col = uint32_t(buf * NC + g * 32 + cofs);
                tc_ld_frag(v0, tmem_base + (uint32_t(quarter * 32) << 16) + col);
                tc_ld_frag(v1, tmem_base + (uint32_t(quarter * 32 + 16) << 16) + col);
                tc_wait_ld();
                if (!masked) stats_block<NB, EP::kFmaExp>(v0, v1, m_run[g], z_run[g], scale2);
                else stats_block_masked<NB>(v0, v1, m_run[g], z_run[g], scale2, t_base, first_masked_key, W, cofs + lq * 2);
            }
            if (i >= kept) {                      // streaming buffer: hand it back to the MMA issuer
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tmem_empty + 8 * buf);
            }
        }

        // merge the running statistics: lanes holding the same columns, then warps, then CTAs
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int jj = 0; jj < 2 * NB; ++jj) {
#pragma unroll
                for (int d = 4; d <= 16; d <<= 1) {
                    const float om = __shfl_xor_sync(0xffffffffu, m_run[g][jj], d);
                    const float oz = __shfl_xor_sync(0xffffffffu, z_run[g][jj], d);
                    merge_stats(m_run[g][jj], z_run[g][jj], om, oz);
                }
                if (lr == 0) wstats[(warp * G + g) * EP::kCols + (jj >> 1) * 8 + lq * 2 + (jj & 1)] = make_float2(m_run[g][jj], z_run[g][jj]);
            }
        epi_sync();
        if (tid < G * 32) {
            const int g = tid >> 5, col = tid & 31;
            const int cs = col / EP::kCols, cl = col % EP::kCols;        // the warp set that holds the column
            float m = kNeg, z = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                const float2 s = wstats[((cs * 8 + w) * G + g) * EP::kCols + cl];
                merge_stats(m, z, s.x, s.y);
            }
            cstats[tid] = make_float2(m, z);
        }
        cluster_arrive();
        cluster_wait();
        if (tid < G * 32) {
            const int g = tid >> 5, col = tid & 31;
            float m, z;
            if (a.lse) {
                // caller-supplied natural-log row sums: use them as (max, sum) = (lse, 1)
                m = (col < W && !skip)
                        ? a.lse[(int64_t(b) * (a.n_kv_heads * G) + h * G + g) * W + col] * 1.4426950408889634f
                        : 0.f;
                z = 1.f;
            } else {
                m = kNeg; z = 0.f;
                for (uint32_t r = 0; r < csize; ++r) {
                    const float2 s = ld_remote_f2(smem_u32(&cstats[tid]), r);
                    merge_stats(m, z, s.x, s.y);
                }
            }
            // weight of 2^(x - m) is 1 / (G (n 2^-m + Z)); fold it and -m into one additive constant
            const float denom = a.n * ex2f(-m) + z;
            cvec[tid] = col < W ? lg2f(a.weight / denom) - m : -INFINITY;
        }
        epi_sync();

        // ---------------------------------- pass 2 ----------------------------------
        float* const out_s = a.score_self + (int64_t(b) * a.n_kv_heads + h) * a.max_len;
        float* const out_c = a.score_cross + (int64_t(b) * a.n_kv_heads + h) * a.max_len;
        const int ndq = *n_dq;
        const uint32_t wmask = W >= 32 ? 0xFFFFFFFFu : ((1u << W) - 1u);

        // this thread's key of tile i is t_of(i); its label is fetched one tile ahead
        auto t_of = [&](int i) { return (i * int(csize) + int(rank)) * kTileKeys + quarter * 32 + lane; };
        uint32_t kmod_next = (group < my_cand && t_of(group) < N) ? modp[t_of(group)] : 0u;
        for (int i = group; i < my_cand; i += 2) {
            const int buf = buf_of(i, 1);
            const int t = t_of(i);
            const uint32_t kmod = kmod_next;
            kmod_next = (i + 2 < my_cand && t_of(i + 2) < N) ? modp[t_of(i + 2)] : 0u;
            mbar_wait(tmem_full + 8 * buf, par_of(i, 1), abort_flag);
            tc_fence_after();
            uint32_t same = 0u;                                            // window columns with the key's label
            for (int q = 0; q < ndq; ++q) same = dq_val[q] == kmod ? dq_mask[q] : same;
            const int delta = t - first_masked_key;                        // column w sees the key iff w >= delta
            const uint32_t vis = delta <= 0 ? wmask : (delta >= 32 ? 0u : (wmask & (0xFFFFFFFFu << delta)));
            const uint32_t add_s = same & vis, add_c = ~same & vis;
            // the row of 32 G logits is read in chunks of 16 columns; the load of the next chunk is in
            // flight while the current one is turned into weights (two accumulators per score)
            float s0 = 0.f, s1 = 0.f, c0 = 0.f, c1 = 0.f;
            float2 p01 = make_float2(0.f, 0.f), p23 = make_float2(0.f, 0.f);   // the plain sums, two-wide
            const uint32_t row_addr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(buf * NC + cofs);
            uint32_t va[16], vb[16];
            tc_ld_row16(va, row_addr);
            // weights of 16 columns: cur = logits, cv = their additive constants, as/ac = which columns count
            auto chunk = [&](const uint32_t (&cur)[16], const float* cvp, uint32_t as, uint32_t ac) {
                const float4* cv = reinterpret_cast<const float4*>(cvp);
                if (want_hist) {
                    // one count per (query head, window row, key) the scores take in: its class is the sum it goes
                    // to, its bin the half-octave of log2(weight).  Lanes with the same (class, bin) are counted
                    // together, one shared-memory add per distinct value.
#pragma unroll 1
                    for (int j = 0; j < 16; ++j) {
                        const bool counted = t < N && (((as | ac) >> j) & 1u);
                        const float e = (fmaf(__uint_as_float(cur[j]), scale2, cvp[j]) + hist_shift) * (1.0f / CSP_HIST_WIDTH);
                        const int bin = min(max(int(floorf(fmaxf(e, 0.f))), 0), kHistBins - 1);
                        const uint32_t key = counted ? uint32_t(((ac >> j) & 1u) * kHistBins + bin) : 0xFFFFu;
                        const uint32_t peers = __match_any_sync(0xffffffffu, key);
                        if (counted && lane == __ffs(peers) - 1) atomicAdd(&whist[key], uint32_t(__popc(peers)));
                    }
                }
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
            };
            // Common case: every window query carries the same label and no column of this tile is hidden.
            // Then a key's weights all go to one of the two sums, chosen once per key, and the columns
            // beyond W add exact zeros (their constant is -inf): plain sums, no per-column selection.
            const bool plain = !want_hist && ndq == 1 && (i * int(csize) + int(rank) + 1) * kTileKeys <= first_masked_key;
            auto chunk_plain = [&](const uint32_t (&cur)[16], const float* cvp) {
                const float4* cv = reinterpret_cast<const float4*>(cvp);
                const float2 sc2 = make_float2(scale2, scale2);
#pragma unroll
                for (int j4 = 0; j4 < 4; ++j4) {
                    const float4 cc = cv[j4];
                    p01 = __fadd2_rn(p01, ex2f2(__ffma2_rn(make_float2(__uint_as_float(cur[j4 * 4 + 0]), __uint_as_float(cur[j4 * 4 + 1])),
                                                           sc2, make_float2(cc.x, cc.y))));
                    const float2 x23 = __ffma2_rn(make_float2(__uint_as_float(cur[j4 * 4 + 2]), __uint_as_float(cur[j4 * 4 + 3])),
                                                  sc2, make_float2(cc.z, cc.w));
                    p23 = __fadd2_rn(p23, (EP::kFmaExp && j4 == 3) ? ex2_fma2(x23) : ex2f2(x23));
                }
            };
            // The thread's columns come in chunks of 16: chunk k sits kStep columns after chunk k - 1 (both
            // halves of every head, or this set's half of every head) and uses bits kShift(k) of the masks.
            // Two chunks per iteration, the load of the next one in flight while one is turned into weights.
            // Fully unrolled for every G: with 7 heads the rolled loop was 4-8 % slower (address arithmetic
            // and a branch per 32 exponentials in a loop that is bound by instruction issue).
            constexpr int kChunks = EP::kSplit ? G : 2 * G;
            constexpr int kStep = EP::kSplit ? 32 : 16;
            const float* const cv_mine = cvec + cofs;
            auto shift_of = [&](int k) { return EP::kSplit ? cofs : (k & 1) * 16; };
            if (plain) {
#pragma unroll
                for (int k = 0; k < kChunks; k += 2) {
                    tc_wait_ld();
                    if (k + 1 < kChunks) tc_ld_row16(vb, row_addr + uint32_t((k + 1) * kStep));
                    chunk_plain(va, cv_mine + k * kStep);
                    if (k + 1 < kChunks) {
                        tc_wait_ld();
                        if (k + 2 < kChunks) tc_ld_row16(va, row_addr + uint32_t((k + 2) * kStep));
                        chunk_plain(vb, cv_mine + (k + 1) * kStep);
                    }
                }
                const float total = (p01.x + p01.y) + (p23.x + p23.y);
                s0 = same ? total : 0.f; s1 = 0.f;
                c0 = same ? 0.f : total; c1 = 0.f;
            } else {
#pragma unroll
                for (int k = 0; k < kChunks; k += 2) {
                    tc_wait_ld();
                    if (k + 1 < kChunks) tc_ld_row16(vb, row_addr + uint32_t((k + 1) * kStep));
                    chunk(va, cv_mine + k * kStep, add_s >> shift_of(k), add_c >> shift_of(k));
                    if (k + 1 < kChunks) {
                        tc_wait_ld();
                        if (k + 2 < kChunks) tc_ld_row16(va, row_addr + uint32_t((k + 2) * kStep));
                        chunk(vb, cv_mine + (k + 1) * kStep, add_s >> shift_of(k + 1), add_c >> shift_of(k + 1));
                    }
                }
            }
            float s = s0 + s1, c = c0 + c1;
            if (i >= kept) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tmem_empty + 8 * buf);
            }
            if (EP::kSplit) {
                // set 1 hands its partial sums to the set-0 warp that holds the same keys (a 64-thread
                // barrier per warp pair); the slot alternates with the iteration, so set 1 can only
                // overwrite it after set 0 has passed the next barrier, i.e. after it has read it
                float2* const slot = xchg + (((i >> 1) & 1) * 2 + group) * 128 + quarter * 32 + lane;
                if (set == 1) *slot = make_float2(s, c);
                asm volatile("bar.sync %0, 64;" ::"r"(2 + group * 4 + quarter) : "memory");
                if (set == 0) { const float2 o = *slot; s += o.x; c += o.y; }
            }
            if (set == 0 && t < N) { out_s[t] = s; out_c[t] = c; }
        }
        if (want_hist) {
            // the warps' counts of this CTA go to the unit's histogram (the CTAs of the cluster add up there)
            epi_sync();
            const uint32_t* const all = reinterpret_cast<const uint32_t*>(base_ptr + sp.hist);
            uint32_t* const dst = a.hist + (int64_t(b) * a.n_kv_heads + h) * 2 * kHistBins;
            for (int j = tid; j < 2 * kHistBins; j += EP::kEpiThreads) {
                uint32_t c = 0;
                for (int w = 0; w < EP::kWarps; ++w) c += all[w * 2 * kHistBins + j];
                if (c) atomicAdd(&dst[j], c);
            }
        }
        if (*abort_flag && tid == 0) atomicOr(a.status, CSP_DEV_TIMEOUT);
    }

    // every warp: give tensor memory back, then keep shared memory alive until the peers are done
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, uint32_t(tmem_cols));
    }
    cluster_arrive();                             // cluster barrier 2
    cluster_wait();
}

template <int NH, int G, bool kHist>
csp_status launch_inst(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s) {
    const int max_tiles = (p.max_len + kTileKeys - 1) / kTileKeys;
    const int units = p.batch * p.n_kv_heads;
    // Two CTAs per SM when (MHA) every CTA can still keep all its tiles in its half of tensor memory.
    bool shared_sm = false;
    const int sms = sm_count();
    int c = pick_cluster(units, max_tiles, TmemPlan<G>::kBufs, sms);
    if (G == 1 && NH <= 2) {
        const int c2 = pick_cluster(units, max_tiles, TmemPlan<G>::kBufsShared, sms);
        if ((max_tiles + c2 - 1) / c2 <= TmemPlan<G>::kBufsShared) { shared_sm = true; c = c2; }
    }
    constexpr bool with_hist = kHist;
    const int fixed = int(tc_smem_plan(NH, G, 0, with_hist).total) + 1024;
    int stages = ((shared_sm ? 113 : 227) * 1024 - fixed) / (NH * kBlockBytes);
    if (stages > 6) stages = 6;
    if (stages < 2) return CSP_ERR_UNSUPPORTED;
    const size_t smem = tc_smem_plan(NH, G, stages, with_hist).total + 1024;
    auto kern = score_tc_kernel<NH, G, kHist>;
    static std::atomic<bool> configured[kMaxDevices];   // per instantiation and device
    if (!raise_smem_limit(kern, 227 * 1024, configured)) return CSP_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(c, p.n_kv_heads, p.batch);
    cfg.blockDim = dim3(EpiPlan<G>::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tmap, a, stages, shared_sm ? 256 : 512) != cudaSuccess) {
        cudaGetLastError();
        return CSP_ERR_CUDA;
    }
    return CSP_OK;
}

// Registers-only loop of base-2 exponentials, for csp_probe_ex2_rate: eight independent chains per thread, either
// on the special-function unit (ex2.approx.ftz.f32, the instruction of the scoring kernels) or through the
// two-wide FMA-pipe evaluation that the G >= 3 kernels use for one pair in eight.
template <bool kFmaPipe>
__global__ void __launch_bounds__(1024) ex2_probe_kernel(int iters, float* sink, size_t sink_elems) {
    float2 x[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] = make_float2(0.1f * float(threadIdx.x & 7) + 0.05f * i, 0.3f + 0.07f * i);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 neg = make_float2(-x[i].x, -x[i].y);      // x <- 2^-x stays in (0.5, 1]
            x[i] = kFmaPipe ? ex2_fma2(neg) : ex2f2(neg);
        }
    }
    const size_t gtid = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (gtid < sink_elems) sink[gtid] = (x[0].x + x[0].y) + (x[1].x + x[1].y) + (x[2].x + x[2].y) + (x[3].x + x[3].y);
}

// the same chain on packed half-precision pairs (ex2.approx.f16x2: two exponentials per instruction), eight packed
// chains per thread
__global__ void __launch_bounds__(1024) ex2_probe_half2_kernel(int iters, float* sink, size_t sink_elems) {
    uint32_t x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = 0x38003400u + uint32_t(threadIdx.x & 7) * 0x00100010u + uint32_t(i);   // halves near 0.5
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t neg = x[i] ^ 0x80008000u;               // x <- 2^-x stays in (0.5, 1]
            asm volatile("ex2.approx.f16x2 %0, %1;" : "=r"(x[i]) : "r"(neg));
        }
    }
    const size_t gtid = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
    uint32_t acc = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) acc ^= x[i];
    if (gtid < sink_elems) sink[gtid] = __uint_as_float(acc & 0x3fffffffu);
}

template <int NH>
csp_status launch_g(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s) {
    switch (a.group) {
        case 1: return a.hist ? launch_inst<NH, 1, true>(p, a, tmap, s) : launch_inst<NH, 1, false>(p, a, tmap, s);
        case 2: return a.hist ? launch_inst<NH, 2, true>(p, a, tmap, s) : launch_inst<NH, 2, false>(p, a, tmap, s);
        case 3: return a.hist ? launch_inst<NH, 3, true>(p, a, tmap, s) : launch_inst<NH, 3, false>(p, a, tmap, s);
        case 4: return a.hist ? launch_inst<NH, 4, true>(p, a, tmap, s) : launch_inst<NH, 4, false>(p, a, tmap, s);
        case 5: return a.hist ? launch_inst<NH, 5, true>(p, a, tmap, s) : launch_inst<NH, 5, false>(p, a, tmap, s);
        case 6: return a.hist ? launch_inst<NH, 6, true>(p, a, tmap, s) : launch_inst<NH, 6, false>(p, a, tmap, s);
        case 7: return a.hist ? launch_inst<NH, 7, true>(p, a, tmap, s) : launch_inst<NH, 7, false>(p, a, tmap, s);
        case 8: return a.hist ? launch_inst<NH, 8, true>(p, a, tmap, s) : launch_inst<NH, 8, false>(p, a, tmap, s);
        default: return CSP_ERR_UNSUPPORTED;
    }
}

}  // namespace

csp_status launch_ex2_probe(int fma_pipe, int iters, float* sink, size_t sink_elems, long long* n_exp, cudaStream_t s) {
    const int blocks = 2 * sm_count();
    if (fma_pipe == 2) ex2_probe_half2_kernel<<<blocks, 1024, 0, s>>>(iters, sink, sink_elems);
    else if (fma_pipe) ex2_probe_kernel<true><<<blocks, 1024, 0, s>>>(iters, sink, sink_elems);
    else ex2_probe_kernel<false><<<blocks, 1024, 0, s>>>(iters, sink, sink_elems);
    if (cudaGetLastError() != cudaSuccess) return CSP_ERR_CUDA;
    *n_exp = (long long)blocks * 1024LL * (fma_pipe == 2 ? 16LL : 8LL) * (long long)iters;
    return CSP_OK;
}

csp_status launch_score_tc(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s) {
    switch (p.head_dim * 2) {
        case 128: return launch_g<1>(p, a, tmap, s);
        case 256: return launch_g<2>(p, a, tmap, s);
        case 512: return launch_g<4>(p, a, tmap, s);
        default: return CSP_ERR_UNSUPPORTED;
    }
}

}  // namespace csp
