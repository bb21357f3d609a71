// Scoring kernel for fp32 caches: window logits (Eq. 5), n-softmax rows (Eq. 7), recent trim,
// head-group mean and the intra/inter query-axis sums (Eq. 1), for one layer.  (bf16 caches take
// the tcgen05 kernel in csp_score_tc.cu; the host entry below builds the K tensor map for both.)
//
// One thread-block cluster of C CTAs owns one (sequence, KV head) unit; 128-key tiles of K are
// dealt round-robin to the CTAs of the cluster.  Each CTA is a TMA producer warp feeding a ring of
// shared-memory stages plus 8 tensor-core consumer warps.
//
//   pass 1  stream the unit's K tiles, logits = K_tile . Q^T on mma.sync (keys on the M axis, the
//           32 window queries of one query head on the N axis), keep a per-thread running
//           (max, sum of 2^(x-max)) per window row; merge over lanes, warps and - through
//           distributed shared memory - over the CTAs of the cluster.
//   pass 2  stream the candidate tiles again (they are L2 hits: a unit's K was just read),
//           recompute the logits, weight = 2^(x-m) / (G (n 2^-m + Z)), add it to the key's intra
//           or inter sum depending on whether query and key labels are equal, reduce over the
//           query axis with quad shuffles and over the query heads of the group through shared
//           memory, write the two score vectors.
//
// Every summation order is fixed, so results are bit-reproducible run to run.
// fp32 products are 3xTF32 (hi/lo split) so that the logits keep fp32 accuracy.
#include <cuda_bf16.h>

#include <mutex>

#include "csp_device.cuh"
#include "csp_internal.cuh"

namespace csp {
namespace {

using namespace dev;

template <int G> struct GroupSplit {           // how the 8 consumer warps are dealt to G query heads
    static constexpr int kWarpsPerHead = G == 1 ? 8 : G == 2 ? 4 : G <= 4 ? 2 : 1;
    static constexpr int kMTilesPerWarp = 8 / kWarpsPerHead;
};

struct SmemPlan {   // byte offsets from the 1024-aligned base
    uint32_t q, part, wstats, cstats, fstats, bars, abort_flag, total;
};
__host__ __device__ inline SmemPlan smem_plan(int nh, int g, int stages) {
    SmemPlan s;
    uint32_t off = uint32_t(stages) * uint32_t(nh) * kBlockBytes;
    s.q = off;          off += uint32_t(nh) * uint32_t(g) * 32u * 128u;
    s.part = off;       off += (g > 1) ? 2u * uint32_t(g) * kTileKeys * 8u : 0u;
    s.wstats = off;     off += kConsumerWarps * 32u * 8u;
    s.cstats = off;     off += uint32_t(g) * 32u * 8u;
    s.fstats = off;     off += uint32_t(g) * 32u * 8u;
    s.bars = off;       off += 2u * 8u * 8u;         // up to 8 stages: full[8], empty[8]
    s.abort_flag = off; off += 16u;
    s.total = off;
    return s;
}

template <typename T, int NH, int G>
__global__ void __launch_bounds__(kThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap tmap, const ScoreArgs a, const int n_stages) {
    constexpr bool kIsF32 = sizeof(T) == 4;
    constexpr int KS = NH * 4;                       // k-steps: 32 bytes of a row each
    constexpr int WPG = GroupSplit<G>::kWarpsPerHead;
    constexpr int MTW = GroupSplit<G>::kMTilesPerWarp;
    constexpr bool kQResident = NH <= 2;
    constexpr uint32_t kStageBytes = NH * kBlockBytes;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const SmemPlan sp = smem_plan(NH, G, n_stages);
    const uint32_t q_s = base + sp.q;
    float2* const part = reinterpret_cast<float2*>(base_ptr + sp.part);
    float2* const wstats = reinterpret_cast<float2*>(base_ptr + sp.wstats);
    float2* const cstats = reinterpret_cast<float2*>(base_ptr + sp.cstats);
    float2* const fstats = reinterpret_cast<float2*>(base_ptr + sp.fstats);
    const uint32_t full_bar = base + sp.bars;
    const uint32_t empty_bar = full_bar + 64;
    volatile int* const abort_flag = reinterpret_cast<volatile int*>(base_ptr + sp.abort_flag);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int h = blockIdx.y, b = blockIdx.z;
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

    constexpr int kActiveWarps = G * WPG;
    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, kActiveWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }

    // ---- stage Q of this KV group: row (g*32 + w), 128-byte column blocks, 16-byte chunks XOR-swizzled
    if (!skip) {
        const uint8_t* qb = static_cast<const uint8_t*>(a.q);
        constexpr int kChunksPerRow = NH * 8;
        for (int i = tid; i < G * 32 * kChunksPerRow; i += kThreads) {
            const int r = i / kChunksPerRow, c = i % kChunksPerRow;
            const int g = r >> 5, w = r & 31;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (w < W) {
                const int64_t e = int64_t(b) * a.q_sb + int64_t(h * G + g) * a.q_sh + int64_t(w) * a.q_st;
                v = *reinterpret_cast<const uint4*>(qb + e * int64_t(sizeof(T)) + c * 16);
            }
            const uint32_t off = uint32_t(c >> 3) * (G * 32 * 128) + uint32_t(r) * 128 + (uint32_t((c & 7) ^ (r & 7)) << 4);
            *reinterpret_cast<uint4*>(base_ptr + sp.q + off) = v;
        }
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // =============================== producer warp ===============================
        cluster_arrive();                         // barrier 1: nothing of ours to publish
        if (lane == 0) {
            const int total = my_all + my_cand;
            for (int it = 0; it < total; ++it) {
                const int slot = it % n_stages;
                const uint32_t round = uint32_t(it / n_stages);
                const int tile = (it < my_all ? it : it - my_all) * int(csize) + int(rank);
                mbar_wait(empty_bar + 8 * slot, (round & 1u) ^ 1u, abort_flag);
                if (*abort_flag) break;
                mbar_expect_tx(full_bar + 8 * slot, kStageBytes);
#pragma unroll
                for (int hb = 0; hb < NH; ++hb)
                    tma_load_4d(base + slot * kStageBytes + hb * kBlockBytes, &tmap, full_bar + 8 * slot,
                                hb * int(128 / sizeof(T)), tile * kTileKeys, h, b);
            }
            if (*abort_flag) {
                // let copies that were issued land before the CTA's shared memory is given up
                const int issued = total < n_stages ? total : n_stages;
                for (int s = 0; s < issued; ++s) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(full_bar + 8 * s, 0) && !mbar_try_wait(full_bar + 8 * s, 1) &&
                           global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
        __syncwarp();
        cluster_wait();
        cluster_arrive();                         // barrier 2: keep shared memory alive for peers
        cluster_wait();
        return;
    }

    // ================================= consumer warps =================================
    const int g_w = warp / WPG;                   // query head (within the group) of this warp
    const int j_w = warp % WPG;                   // which m-tiles of a key tile it takes
    const bool active = warp < kActiveWarps;
    const int lq = lane & 3, lr = lane >> 2;

    // resident B fragments (the 32 window queries of head g_w)
    uint32_t bq[kQResident ? KS : 1][4][2];
    const int mid = lane >> 3;
    auto q_frag_addr = [&](int ks, int pair) -> uint32_t {   // ldmatrix.x4: n-tiles 2*pair, 2*pair+1
        const int row = g_w * 32 + (2 * pair + (mid >> 1)) * 8 + (lane & 7);
        const int chunk = (ks & 3) * 2 + (mid & 1);
        return q_s + uint32_t(ks >> 2) * (G * 32 * 128) + uint32_t(row) * 128 + (uint32_t(chunk ^ (row & 7)) << 4);
    };
    if constexpr (kQResident) if (active) {
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
#pragma unroll
            for (int pr = 0; pr < 2; ++pr) {
                uint32_t r[4];
                ldmatrix_x4(r, q_frag_addr(ks, pr));
                bq[ks][2 * pr][0] = r[0]; bq[ks][2 * pr][1] = r[1];
                bq[ks][2 * pr + 1][0] = r[2]; bq[ks][2 * pr + 1][1] = r[3];
            }
    }

    // logits of one 16-key m-tile against the 32 queries of head g_w: acc[nt][0..3]
    auto tile_logits = [&](uint32_t stage_addr, int mt, float (&acc)[4][4]) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
        const int row = mt * 16 + (mid & 1) * 8 + (lane & 7);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            const int chunk = (ks & 3) * 2 + (mid >> 1);
            uint32_t af[4];
            ldmatrix_x4(af, stage_addr + uint32_t(ks >> 2) * kBlockBytes + uint32_t(row) * 128 +
                                (uint32_t(chunk ^ (row & 7)) << 4));
            uint32_t bf[4][2];
            if constexpr (kQResident) {
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) { bf[nt][0] = bq[ks][nt][0]; bf[nt][1] = bq[ks][nt][1]; }
            } else {
#pragma unroll
                for (int pr = 0; pr < 2; ++pr) {
                    uint32_t r[4];
                    ldmatrix_x4(r, q_frag_addr(ks, pr));
                    bf[2 * pr][0] = r[0]; bf[2 * pr][1] = r[1];
                    bf[2 * pr + 1][0] = r[2]; bf[2 * pr + 1][1] = r[3];
                }
            }
            if constexpr (kIsF32) {
                uint32_t ah[4], al[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) split_tf32(af[e], ah[e], al[e]);
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    uint32_t bh0, bl0, bh1, bl1;
                    split_tf32(bf[nt][0], bh0, bl0);
                    split_tf32(bf[nt][1], bh1, bl1);
                    mma_tf32(acc[nt], al, bh0, bh1);
                    mma_tf32(acc[nt], ah, bl0, bl1);
                    mma_tf32(acc[nt], ah, bh0, bh1);
                }
            } else {
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) mma_bf16(acc[nt], af, bf[nt][0], bf[nt][1]);
            }
        }
    };

    const float scale2 = a.scale_log2;
    const int first_masked_key = L - W;           // keys beyond this may be hidden from some row
    int it = 0;                                   // ring sequence number, shared by both passes

    // ---------------------------------- pass 1 ----------------------------------
    float m_run[8], z_run[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) { m_run[jj] = kNeg; z_run[jj] = 0.f; }

    for (int i = 0; i < my_all; ++i, ++it) {
        const int slot = it % n_stages;
        const int tile = i * int(csize) + int(rank);
        if (!active) continue;
        mbar_wait(full_bar + 8 * slot, uint32_t(it / n_stages) & 1u, abort_flag);
        const uint32_t stage_addr = base + slot * kStageBytes;
        const bool masked = (tile + 1) * kTileKeys > first_masked_key;
#pragma unroll
        for (int mi = 0; mi < MTW; ++mi) {
            const int mt = j_w + mi * WPG;
            float acc[4][4];
            tile_logits(stage_addr, mt, acc);
            const int t0 = tile * kTileKeys + mt * 16 + lr;
            if (!masked) {
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int jj = nt * 2 + e;
                        const float x0 = acc[nt][e] * scale2, x1 = acc[nt][2 + e] * scale2;
                        const float mx = fmaxf(x0, x1);
                        if (mx > m_run[jj] + kLazy) { z_run[jj] *= ex2f(m_run[jj] - mx); m_run[jj] = mx; }
                        z_run[jj] += ex2f(x0 - m_run[jj]) + ex2f(x1 - m_run[jj]);
                    }
            } else {
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int jj = nt * 2 + e;
                        const int col = nt * 8 + lq * 2 + e;
                        const bool v0 = col < W && t0 <= first_masked_key + col;       // key <= query position
                        const bool v1 = col < W && t0 + 8 <= first_masked_key + col;
                        const float x0 = v0 ? acc[nt][e] * scale2 : kNeg;
                        const float x1 = v1 ? acc[nt][2 + e] * scale2 : kNeg;
                        const float mx = fmaxf(x0, x1);
                        if (mx > m_run[jj] + kLazy) { z_run[jj] *= ex2f(m_run[jj] - mx); m_run[jj] = mx; }
                        z_run[jj] += (v0 ? ex2f(x0 - m_run[jj]) : 0.f) + (v1 ? ex2f(x1 - m_run[jj]) : 0.f);
                    }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar + 8 * slot);
    }

    // merge the running statistics: lanes holding the same columns, then warps, then CTAs
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) {
#pragma unroll
        for (int d = 4; d <= 16; d <<= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, m_run[jj], d);
            const float oz = __shfl_xor_sync(0xffffffffu, z_run[jj], d);
            merge_stats(m_run[jj], z_run[jj], om, oz);
        }
    }
    if (lr == 0) {
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const int col = (jj >> 1) * 8 + lq * 2 + (jj & 1);
            wstats[warp * 32 + col] = make_float2(m_run[jj], z_run[jj]);
        }
    }
    consumer_sync();
    if (tid < G * 32) {
        const int g = tid >> 5, col = tid & 31;
        float m = kNeg, z = 0.f;
#pragma unroll
        for (int w = 0; w < WPG; ++w) {
            const float2 s = wstats[(g * WPG + w) * 32 + col];
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
        // weight of one unit of 2^(x-m): 1 / (G (n 2^-m + Z)); padding rows of the window get 0
        const float denom = a.n * ex2f(-m) + z;
        fstats[tid] = col < W ? make_float2(m, a.weight / denom) : make_float2(0.f, 0.f);
    }
    consumer_sync();

    // ---------------------------------- pass 2 ----------------------------------
    const uint8_t* modp = a.modality + int64_t(b) * a.mod_sb + int64_t(h) * a.mod_sh;
    uint32_t qmod[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) {
        const int col = (jj >> 1) * 8 + lq * 2 + (jj & 1);
        qmod[jj] = (col < W && !skip) ? modp[L - W + col] : 0u;
    }
    float* const out_s = a.score_self + (int64_t(b) * a.n_kv_heads + h) * a.max_len;
    float* const out_c = a.score_cross + (int64_t(b) * a.n_kv_heads + h) * a.max_len;

    for (int i = 0; i < my_cand; ++i, ++it) {
        const int slot = it % n_stages;
        const int tile = i * int(csize) + int(rank);
        float2* const pbuf = part + (i & 1) * (G * kTileKeys);
        if (active) {
            mbar_wait(full_bar + 8 * slot, uint32_t(it / n_stages) & 1u, abort_flag);
            const uint32_t stage_addr = base + slot * kStageBytes;
            const bool masked = (tile + 1) * kTileKeys > first_masked_key;
#pragma unroll
            for (int mi = 0; mi < MTW; ++mi) {
                const int mt = j_w + mi * WPG;
                const int t0 = tile * kTileKeys + mt * 16 + lr, t1 = t0 + 8;
                const uint32_t km0 = t0 < N ? modp[t0] : 0u, km1 = t1 < N ? modp[t1] : 0u;
                float acc[4][4];
                tile_logits(stage_addr, mt, acc);
                float s0 = 0.f, c0 = 0.f, s1 = 0.f, c1 = 0.f;
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int jj = nt * 2 + e;
                        const int col = nt * 8 + lq * 2 + e;
                        const float2 st = fstats[g_w * 32 + col];
                        float p0 = ex2f(fmaf(acc[nt][e], scale2, -st.x)) * st.y;
                        float p1 = ex2f(fmaf(acc[nt][2 + e], scale2, -st.x)) * st.y;
                        if (masked) {
                            if (!(t0 <= first_masked_key + col)) p0 = 0.f;
                            if (!(t1 <= first_masked_key + col)) p1 = 0.f;
                        }
                        if (qmod[jj] == km0) s0 += p0; else c0 += p0;
                        if (qmod[jj] == km1) s1 += p1; else c1 += p1;
                    }
                // sum over the query axis: the 4 lanes of a quad hold the 32 columns of a row
#pragma unroll
                for (int d = 1; d <= 2; d <<= 1) {
                    s0 += __shfl_xor_sync(0xffffffffu, s0, d); c0 += __shfl_xor_sync(0xffffffffu, c0, d);
                    s1 += __shfl_xor_sync(0xffffffffu, s1, d); c1 += __shfl_xor_sync(0xffffffffu, c1, d);
                }
                if (lq == 0) {
                    if (G == 1) {
                        if (t0 < N) { out_s[t0] = s0; out_c[t0] = c0; }
                        if (t1 < N) { out_s[t1] = s1; out_c[t1] = c1; }
                    } else {
                        pbuf[g_w * kTileKeys + mt * 16 + lr] = make_float2(s0, c0);
                        pbuf[g_w * kTileKeys + mt * 16 + lr + 8] = make_float2(s1, c1);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar + 8 * slot);
        }
        if (G > 1) {
            consumer_sync();                      // partials of all query heads are in place
            if (tid < kTileKeys) {
                const int t = tile * kTileKeys + tid;
                float s = 0.f, c = 0.f;
#pragma unroll
                for (int g = 0; g < G; ++g) { const float2 v = pbuf[g * kTileKeys + tid]; s += v.x; c += v.y; }
                if (t < N) { out_s[t] = s; out_c[t] = c; }
            }
        }
    }

    if (*abort_flag && tid == 0) atomicOr(a.status, CSP_DEV_TIMEOUT);
    cluster_arrive();                             // barrier 2: peers may still be reading cstats
    cluster_wait();
}

// mean over the KV heads of per-head partial sums (each already weighted 1/Hq), written to every head
__global__ void head_mean_kernel(const float* __restrict__ part_self, const float* __restrict__ part_cross,
                                 float* __restrict__ score_self, float* __restrict__ score_cross,
                                 const int32_t* __restrict__ seq_lens, int n_kv_heads, int max_len, int recent,
                                 int window) {
    const int b = blockIdx.y;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int L = seq_lens[b];
    if (L < window || L > max_len || t >= L - recent) return;
    float s = 0.f, c = 0.f;
    for (int h = 0; h < n_kv_heads; ++h) {
        s += part_self[(int64_t(b) * n_kv_heads + h) * max_len + t];
        c += part_cross[(int64_t(b) * n_kv_heads + h) * max_len + t];
    }
    for (int h = 0; h < n_kv_heads; ++h) {
        score_self[(int64_t(b) * n_kv_heads + h) * max_len + t] = s;
        score_cross[(int64_t(b) * n_kv_heads + h) * max_len + t] = c;
    }
}

// Jensen-Shannon divergence (nats) between the intra and the inter histogram of every unit (blocks 0 .. units-1)
// and of their sums over all units (block `units`): 1/2 KL(P || M) + 1/2 KL(Q || M), M = (P + Q) / 2, with P and Q
// normalised to sum 1 and 0 log 0 = 0; NaN when either histogram is empty.  One thread per bin.
__global__ void __launch_bounds__(CSP_HIST_BINS) hist_js_kernel(const uint32_t* __restrict__ hist, int units,
                                                                float* __restrict__ js, float* __restrict__ js_all) {
    constexpr int NB = CSP_HIST_BINS;
    __shared__ double red[2][NB];
    const int j = threadIdx.x, u = blockIdx.x;
    const bool pooled = u == units;
    if ((pooled && !js_all) || (!pooled && !js)) return;
    double cp = 0.0, cq = 0.0;
    if (pooled) {
        for (int v = 0; v < units; ++v) {
            cp += double(hist[(int64_t(v) * 2) * NB + j]);
            cq += double(hist[(int64_t(v) * 2 + 1) * NB + j]);
        }
    } else {
        cp = double(hist[(int64_t(u) * 2) * NB + j]);
        cq = double(hist[(int64_t(u) * 2 + 1) * NB + j]);
    }
    auto block_sums = [&](double x, double y, double& sx, double& sy) {     // fixed-order tree over the bins
        red[0][j] = x; red[1][j] = y;
        __syncthreads();
        for (int d = NB / 2; d > 0; d >>= 1) {
            if (j < d) { red[0][j] += red[0][j + d]; red[1][j] += red[1][j + d]; }
            __syncthreads();
        }
        sx = red[0][0]; sy = red[1][0];
        __syncthreads();
    };
    double sp, sq;
    block_sums(cp, cq, sp, sq);
    double term = 0.0, unused = 0.0, total, dummy;
    if (sp > 0.0 && sq > 0.0) {
        const double pj = cp / sp, qj = cq / sq, mj = 0.5 * (pj + qj);
        if (pj > 0.0) term += 0.5 * pj * log(pj / mj);
        if (qj > 0.0) term += 0.5 * qj * log(qj / mj);
    }
    block_sums(term, unused, total, dummy);
    if (j == 0) {
        const float r = (sp > 0.0 && sq > 0.0) ? float(total) : __int_as_float(0x7fc00000);
        if (pooled) *js_all = r; else js[u] = r;
    }
}

// ---- host side --------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

template <typename T, int NH, int G>
csp_status launch_inst(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s) {
    const int fixed = int(smem_plan(NH, G, 0).total) + 1024;
    int stages = (227 * 1024 - fixed) / (NH * kBlockBytes);
    if (stages > 6) stages = 6;
    if (stages < 2) return CSP_ERR_UNSUPPORTED;
    const size_t smem = smem_plan(NH, G, stages).total + 1024;
    auto kern = score_kernel<T, NH, G>;
    static std::atomic<bool> configured[kMaxDevices];   // per instantiation and device
    if (!raise_smem_limit(kern, 227 * 1024, configured)) return CSP_ERR_CUDA;
    const int max_tiles = (p.max_len + kTileKeys - 1) / kTileKeys;
    const int c = pick_cluster(p.batch * p.n_kv_heads, max_tiles, 0, sm_count());
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(c, p.n_kv_heads, p.batch);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tmap, a, stages) != cudaSuccess) { cudaGetLastError(); return CSP_ERR_CUDA; }
    return CSP_OK;
}

template <typename T, int NH>
csp_status launch_g(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s) {
    switch (a.group) {
        case 1: return launch_inst<T, NH, 1>(p, a, tmap, s);
        case 2: return launch_inst<T, NH, 2>(p, a, tmap, s);
        case 3: return launch_inst<T, NH, 3>(p, a, tmap, s);
        case 4: return launch_inst<T, NH, 4>(p, a, tmap, s);
        case 5: return launch_inst<T, NH, 5>(p, a, tmap, s);
        case 6: return launch_inst<T, NH, 6>(p, a, tmap, s);
        case 7: return launch_inst<T, NH, 7>(p, a, tmap, s);
        case 8: return launch_inst<T, NH, 8>(p, a, tmap, s);
        default: return CSP_ERR_UNSUPPORTED;
    }
}

template <typename T>
csp_status launch_t(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s) {
    const int row_bytes = p.head_dim * int(sizeof(T));
    switch (row_bytes) {
        case 128: return launch_g<T, 1>(p, a, tmap, s);
        case 256: return launch_g<T, 2>(p, a, tmap, s);
        case 512: return launch_g<T, 4>(p, a, tmap, s);
        default: return CSP_ERR_UNSUPPORTED;
    }
}

// order[r] = the sequence with the r-th longest valid length (ties: lower index first).  The scoring
// kernels take sequences in this order, longest first, so that a ragged batch does not end with one
// long unit running alone.
__global__ void length_order_kernel(const int32_t* __restrict__ seq_lens, int batch, int max_len,
                                    int32_t* __restrict__ order) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= batch) return;
    auto len = [&](int i) { const int L = seq_lens[i]; return (L < 0 || L > max_len) ? 0 : L; };
    const int Lt = len(t);
    int r = 0;
    for (int j = 0; j < batch; ++j) {
        const int Lj = len(j);
        r += (Lj > Lt || (Lj == Lt && j < t)) ? 1 : 0;
    }
    order[r] = t;
}

}  // namespace

bool make_cache_tensor_map(CUtensorMap* map, const csp_tensor& t, int dtype, int head_dim, int rows, int heads,
                           int batch, int box_rows) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return false;
    const uint64_t es = dtype == CSP_F32 ? 4 : 2;
    // sizes of 1 carry no usable stride: give them a legal one
    const uint64_t st = uint64_t(t.stride_t) * es;
    const uint64_t sh = heads > 1 ? uint64_t(t.stride_h) * es : st * uint64_t(rows);
    const uint64_t sb = batch > 1 ? uint64_t(t.stride_b) * es : sh * uint64_t(heads);
    if (t.stride_t < head_dim || (st % 16) || (sh % 16) || (sb % 16) || (uintptr_t(t.ptr) % 16)) return false;
    const cuuint64_t dims[4] = {cuuint64_t(head_dim), cuuint64_t(rows), cuuint64_t(heads), cuuint64_t(batch)};
    const cuuint64_t strides[3] = {st, sh, sb};
    const cuuint32_t box[4] = {cuuint32_t(128 / es), cuuint32_t(box_rows), 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return encode(map, dtype == CSP_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, t.ptr,
                  dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

csp_status launch_score(const csp_params& p, const ScoreArgs& a_in, const csp_tensor& k, cudaStream_t s,
                        const csp_pages* pages) {
    ScoreArgs a = a_in;
    a.page_table = nullptr; a.max_pages = 0; a.tiles_per_page = 1; a.n_pages = 0;
    // a paged cache: the tensor map describes the page pool [pages, heads, page_rows, head_dim]
    const int map_rows = pages ? pages->page_rows : p.max_len;
    const int map_outer = pages ? pages->n_pages : p.batch;
    if (pages) {
        if (p.dtype != CSP_BF16 || p.head_reduce != CSP_HEADS_PER_KV) return CSP_ERR_UNSUPPORTED;
        a.page_table = pages->page_table; a.max_pages = pages->max_pages; a.tiles_per_page = pages->page_rows / kTileKeys;
        a.n_pages = pages->n_pages;
    }
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return CSP_ERR_CUDA;
    const uint64_t es = p.dtype == CSP_F32 ? 4 : 2;
    const uint64_t row_bytes = uint64_t(p.head_dim) * es;
    // sizes of 1 carry no usable stride: give them a legal one
    const uint64_t st = uint64_t(k.stride_t) * es;
    const uint64_t sh = p.n_kv_heads > 1 ? uint64_t(k.stride_h) * es : st * uint64_t(map_rows);
    const uint64_t sb = map_outer > 1 ? uint64_t(k.stride_b) * es : sh * uint64_t(p.n_kv_heads);
    if (k.stride_t < p.head_dim || (st % 16) || (sh % 16) || (sb % 16) || (uintptr_t(k.ptr) % 16))
        return CSP_ERR_UNSUPPORTED;
    CUtensorMap tmap;
    const cuuint64_t dims[4] = {cuuint64_t(p.head_dim), cuuint64_t(map_rows), cuuint64_t(p.n_kv_heads),
                                cuuint64_t(map_outer)};
    const cuuint64_t strides[3] = {st, sh, sb};
    const cuuint32_t box[4] = {cuuint32_t(128 / es), cuuint32_t(kTileKeys), 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    (void)row_bytes;
    const CUresult r = encode(&tmap, p.dtype == CSP_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                              4, k.ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return CSP_ERR_CUDA;      // strides and alignment were checked above: the driver call itself failed
    if (p.dtype == CSP_F32) return launch_t<float>(p, a, tmap, s);
    // several sequences and more CTAs than fit on the GPU at once (up to 8 per unit; clusters of 8 occupy
    // about 13/16 of the SMs, 120 of a B200's 148): take the sequences longest first
    const int max_tiles = (p.max_len + kTileKeys - 1) / kTileKeys;
    const long long units = (long long)p.batch * p.n_kv_heads;
    const int sms = sm_count();
    if (p.batch >= 2 && p.batch <= 4096 && (units > sms || units * (max_tiles < 8 ? max_tiles : 8) > sms * 13 / 16)) {
        length_order_kernel<<<(p.batch + 255) / 256, 256, 0, s>>>(a.seq_lens, p.batch, p.max_len, a.order_buf);
        if (cudaGetLastError() != cudaSuccess) return CSP_ERR_CUDA;
        a.order = a.order_buf;
    }
    // many MHA units: resident clusters that stream unit after unit; otherwise one cluster per unit
    bool taken = false;
    const csp_status ps = launch_score_persist(p, a, tmap, s, &taken);
    if (ps != CSP_OK || taken) return ps;
    return launch_score_tc(p, a, tmap, s);
}

csp_status launch_hist_js(const csp_params& p, const uint32_t* hist, float* js, float* js_all, cudaStream_t s) {
    const int units = p.batch * p.n_kv_heads;
    if (!js && !js_all) return CSP_OK;
    hist_js_kernel<<<units + 1, CSP_HIST_BINS, 0, s>>>(hist, units, js, js_all);
    return cudaGetLastError() == cudaSuccess ? CSP_OK : CSP_ERR_CUDA;
}

csp_status launch_head_mean(const csp_params& p, const float* part_self, const float* part_cross,
                            float* score_self, float* score_cross, const int32_t* seq_lens, cudaStream_t s) {
    const dim3 grid((p.max_len + 255) / 256, p.batch);
    head_mean_kernel<<<grid, 256, 0, s>>>(part_self, part_cross, score_self, score_cross, seq_lens,
                                          p.n_kv_heads, p.max_len, p.recent, p.window);
    return cudaGetLastError() == cudaSuccess ? CSP_OK : CSP_ERR_CUDA;
}

}  // namespace csp
