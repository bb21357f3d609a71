// Decode attention over a pruned cache with the n-softmax normaliser (Section 3.3, Eq. 6-7): one new query
// per head attends to the n_rows[b, h_kv] rows that a prune left,
//   out[b, h_q, :] = sum_t  e^{o_t} / (n + sum_j e^{o_j})  v[b, h_kv, t, :],   o_t = scale <q, k_t>.
//
// The work is one pass over K and V: HBM-bound (512 bytes per cached row and KV head at d = 128).  The rows of a
// (sequence, KV head) unit are split into work items so that a small batch still fills the GPU; one CTA per SM
// stays resident and walks over items; every item leaves an un-normalised partial result (reference exponent
// m, sum l, weighted value sum) and a second small kernel merges the partials and divides by n 2^-m + l.
//
// Inside a CTA
//   warp 4      one thread streams 64-row tiles of K and V with TMA (128-byte swizzle, no multicast) through a
//               ring of six shared-memory stages, bounded waits on full/empty mbarriers; it runs ahead into the
//               next item, so the stream does not drain between items
//   warps 0-3   each owns 16 rows of every tile.  The G query heads that share the KV head are the M rows of a
//               bf16 m16n8k16 mma (padded to 16): S = Q K^T from ldmatrix fragments, streaming softmax in the
//               base-2 domain with a lazily raised reference, then P V with P split into a bf16 head and a bf16
//               remainder (two mma per fragment) so that the weights keep fp32-like accuracy.
// This is a skinny contraction (at most 8 query rows per key): the legacy warp-level mma is ample for an
// HBM-bound stream, and tensor memory would add nothing.
#include <mutex>

#include "csp_device.cuh"
#include "csp_internal.cuh"

namespace csp {
namespace {
using namespace dev;

constexpr int kDecTile = 64;                       // rows per stage
constexpr int kDecWarps = 4;                       // consumer warps, 16 rows of every tile each
constexpr int kDecThreads = 32 * (kDecWarps + 1);
constexpr int kDecStages = 6;                      // 32 KB each at d = 128: one resident CTA per SM
constexpr int kDecBlock = kDecTile * 128;          // bytes of one 64-column block of a tile

struct DecodeArgs {
    const void* q; int64_t q_sb, q_sh;             // element strides of [B, Hq, d]
    const int32_t* n_rows;                         // [B, Hkv]
    float* partial;                                // [units, splits, G, d + 2]
    float* out;                                    // [B, Hq, d]
    int32_t* status;
    int32_t* next_item;                            // work counter in the status area: zero between calls
    int32_t n_kv_heads, group, head_dim, capacity, splits, tiles_per_split;
    float n, scale_log2;
    // csp_decode_step only: the step's logits are kept so that its n-softmax weights can be added to the running
    // intra / inter sums of Eq. 1 once the row's normaliser is known
    float* logits;                                 // [units, G, capacity]: o scale log2(e), or null
    const uint8_t* modality; int64_t mod_sb, mod_sh;
    const uint8_t* query_label;                    // [B]
    float* acc_self; float* acc_cross;             // [units, capacity]
    int32_t first_step;
    // paged cache: rows [i page_rows, (i + 1) page_rows) of sequence b are page page_table[b * max_pages + i] of the
    // pool the tensor maps describe; null for a dense cache
    const int32_t* page_table; int32_t max_pages, page_rows, n_pages;
};

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A B with A = (a0, 0, a2, 0): rows 8-15 of the 16-row operand are padding
__device__ __forceinline__ void mma_rows8(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
// two floats -> packed bf16 pair (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// barrier over the consumer threads (barrier 1) that also tells everyone whether any of them saw `pred`
__device__ __forceinline__ bool consumers_any(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "barrier.cta.red.or.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"(uint32_t(pred)), "n"(32 * kDecWarps) : "memory");
    return r != 0;
}

template <int NH, bool kKeepLogits>   // head_dim = 64 NH; kKeepLogits: also write every logit to a.logits
__global__ void __launch_bounds__(kDecThreads, 1)
decode_attn_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const DecodeArgs a, const int n_items) {
    constexpr int D = 64 * NH;
    constexpr int KS = D / 16;                     // k-steps of S = Q K^T
    constexpr int NT = D / 8;                      // 8-column tiles of the output
    constexpr uint32_t kTileBytes = NH * kDecBlock;           // K (or V) of one stage
    constexpr uint32_t kStageBytes = 2 * kTileBytes;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    float* const merge = reinterpret_cast<float*>(base_ptr + kDecStages * kStageBytes);     // [warp][8][D + 2]
    const uint32_t full_bar = base + kDecStages * kStageBytes + kDecWarps * 8 * (D + 2) * 4;   // then: abort flag, item queue
    const uint32_t empty_bar = full_bar + 8 * kDecStages;
    volatile int* const abort_flag = reinterpret_cast<volatile int*>(base_ptr + kDecStages * kStageBytes +
                                                                     kDecWarps * 8 * (D + 2) * 4 + 16 * kDecStages);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // Work item = (unit, split): a contiguous range of 64-row tiles of one (sequence, KV head).  The CTA is
    // resident; its producer thread draws items from a global counter (so ragged row counts balance by
    // themselves), tells the consumers which item the next tiles belong to through a small queue in shared
    // memory, and runs ahead into the next item while the consumers finish the current one.
    constexpr int kQueue = 8;                      // > stages: the producer is at most kDecStages items ahead
    volatile int* const item_q = abort_flag + 1;
    struct Item { int u, b, h, sp, rows, tile0, n_tiles; };
    auto item_of = [&](int w) {
        Item x;
        x.u = w / a.splits; x.sp = w % a.splits;
        x.b = x.u / a.n_kv_heads; x.h = x.u % a.n_kv_heads;
        int rows = a.n_rows[x.u];
        rows = rows < 0 ? 0 : (rows > a.capacity ? a.capacity : rows);
        x.rows = rows;
        const int tiles = (rows + kDecTile - 1) / kDecTile;
        x.tile0 = x.sp * a.tiles_per_split;
        const int t1 = min(tiles, x.tile0 + a.tiles_per_split);
        x.n_tiles = t1 > x.tile0 ? t1 - x.tile0 : 0;       // 0: nothing for this split, the merge kernel skips it too
        return x;
    };

    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kDecStages; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, kDecWarps); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    if (warp == kDecWarps) {
        // =============================== TMA producer ===============================
        if (lane == 0) {
            int it = 0, j = 0;
            while (!*abort_flag) {
                const int w = atomicAdd(a.next_item, 1);
                if (w >= n_items) break;
                const Item x = item_of(w);
                if (x.n_tiles == 0) continue;
                for (int i = 0; i < x.n_tiles; ++i, ++it) {
                    const int s = it % kDecStages;
                    mbar_wait(empty_bar + 8 * s, (uint32_t(it / kDecStages) & 1u) ^ 1u, abort_flag);
                    if (*abort_flag) break;
                    if (i == 0) item_q[j % kQueue] = w;     // published by the arrive below (release)
                    mbar_expect_tx(full_bar + 8 * s, kStageBytes);
                    int row = (x.tile0 + i) * kDecTile, outer = x.b;
                    if (a.page_table) {
                        // a page number outside the pool becomes an out-of-range coordinate: zeros arrive, nothing faults
                        outer = a.page_table[int64_t(x.b) * a.max_pages + row / a.page_rows];
                        if (outer < 0 || outer >= a.n_pages) { atomicOr(a.status, CSP_DEV_BAD_LEN); outer = a.n_pages; }
                        row %= a.page_rows;
                    }
#pragma unroll
                    for (int hb = 0; hb < NH; ++hb) {
                        tma_load_4d(base + s * kStageBytes + hb * kDecBlock, &tmap_k, full_bar + 8 * s, hb * 64, row, x.h, outer);
                        tma_load_4d(base + s * kStageBytes + kTileBytes + hb * kDecBlock, &tmap_v, full_bar + 8 * s, hb * 64, row, x.h, outer);
                    }
                }
                ++j;
            }
            if (!*abort_flag) {
                // end marker: one more phase of the next stage's barrier, without data
                const int s = it % kDecStages;
                mbar_wait(empty_bar + 8 * s, (uint32_t(it / kDecStages) & 1u) ^ 1u, abort_flag);
                item_q[j % kQueue] = -1;
                mbar_arrive(full_bar + 8 * s);
            }
            if (*abort_flag) {
                // let copies that were issued land before the CTA's shared memory is given up
                for (int s = 0; s < kDecStages; ++s) {
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(full_bar + 8 * s, 0) && !mbar_try_wait(full_bar + 8 * s, 1) &&
                           global_ns() - t0 < kWaitLimitNs / 8) {}
                }
            }
        }
    } else {
        // =============================== consumer warps ===============================
        const int g = lane >> 2, qd = lane & 3;    // this thread's query row and column pair
        const int G = a.group;
        // ldmatrix row addresses: lane l supplies row (l % 8) of matrix (l / 8)
        const int kr = warp * 16 + ((lane >> 4) << 3) + (lane & 7);      // K: matrices 2,3 are the second 8 rows
        const int kc = (lane >> 3) & 1;                                  //    matrices 1,3 the second 8 columns
        const int vr = warp * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);  // V: matrices 1,3 are the second 8 rows
        const int vc = lane >> 4;                                        //    matrices 2,3 the next 8 columns
        auto consumers_sync = [] { asm volatile("bar.sync 1, %0;" ::"n"(32 * kDecWarps) : "memory"); };
        int it = 0;
        for (int j = 0;; ++j) {
            // the first tile of the next item (or the end marker) tells which item it is
            const bool ok = mbar_wait(full_bar + 8 * (it % kDecStages), uint32_t(it / kDecStages) & 1u, abort_flag);
            const int w = ok ? item_q[j % kQueue] : -1;
            if (consumers_any(w < 0)) break;       // end of work, or a wait gave up: all consumers leave together
            const Item x = item_of(w);
            const int rows = x.rows;
            // Q fragments: row g, columns 16 ks + 2 qd + {0,1} and + 8
            uint32_t qa0[KS], qa2[KS];
            {
                const uint16_t* qrow = static_cast<const uint16_t*>(a.q) + int64_t(x.b) * a.q_sb + int64_t(x.h * G + g) * a.q_sh;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    qa0[ks] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * qd) : 0u;
                    qa2[ks] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * qd) : 0u;
                }
            }
            float acc[NT][4];
#pragma unroll
            for (int t = 0; t < NT; ++t) { acc[t][0] = acc[t][1] = acc[t][2] = acc[t][3] = 0.f; }
            float m_run = kNeg, l_run = 0.f;       // reference exponent of row g, this thread's share of its sum

            for (int i = 0; i < x.n_tiles; ++i, ++it) {
                const int s = it % kDecStages;
                mbar_wait(full_bar + 8 * s, uint32_t(it / kDecStages) & 1u, abort_flag);
                const uint32_t k_s = base + s * kStageBytes, v_s = k_s + kTileBytes;
                const int row_t = (x.tile0 + i) * kDecTile;              // first row of the tile
                const int row_w = row_t + warp * 16;                     // first row of this warp's slice
                if (row_w + 16 > rows) {
                    // Rows past the end hold whatever the cache holds: their weights are zero, but zero times a
                    // non-finite value is not, so clear this warp's value rows beyond the end.
                    for (int j = lane; j < 16 * NH * 8; j += 32) {
                        const int r = warp * 16 + j / (NH * 8), c = j % (NH * 8);
                        if (row_t + r >= rows)
                            *reinterpret_cast<uint4*>(base_ptr + (v_s - base) + (c >> 3) * kDecBlock + r * 128 +
                                                      (((c & 7) ^ (r & 7)) << 4)) = make_uint4(0, 0, 0, 0);
                    }
                    __syncwarp();
                }
                // ---- S = Q K^T for 16 rows: two 8-row tiles
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int chunk = ks * 2 + kc;
                    uint32_t kb[4];
                    ldsm_x4(kb, k_s + (chunk >> 3) * kDecBlock + kr * 128 + (((chunk & 7) ^ (kr & 7)) << 4));
                    mma_rows8(s0, qa0[ks], qa2[ks], kb[0], kb[1]);
                    mma_rows8(s1, qa0[ks], qa2[ks], kb[2], kb[3]);
                }
                // ---- streaming softmax of row g over rows row_w + {2 qd, 2 qd + 1, 8 + 2 qd, 9 + 2 qd}
                const int r0 = row_w + 2 * qd;
                float xs[4] = {r0 < rows ? s0[0] * a.scale_log2 : kNeg, r0 + 1 < rows ? s0[1] * a.scale_log2 : kNeg,
                               r0 + 8 < rows ? s1[0] * a.scale_log2 : kNeg, r0 + 9 < rows ? s1[1] * a.scale_log2 : kNeg};
                if (kKeepLogits && g < G) {
                    float* const lrow = a.logits + (int64_t(x.u) * G + g) * a.capacity;
                    if (r0 < rows) lrow[r0] = xs[0];
                    if (r0 + 1 < rows) lrow[r0 + 1] = xs[1];
                    if (r0 + 8 < rows) lrow[r0 + 8] = xs[2];
                    if (r0 + 9 < rows) lrow[r0 + 9] = xs[3];
                }
                float mx = fmaxf(fmaxf(xs[0], xs[1]), fmaxf(xs[2], xs[3]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                if (mx > m_run + kLazy) {          // same decision in the four lanes of a row
                    const float alpha = ex2f(m_run - mx);
                    l_run *= alpha;
#pragma unroll
                    for (int t = 0; t < NT; ++t) { acc[t][0] *= alpha; acc[t][1] *= alpha; }
                    m_run = mx;
                }
                float p[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) p[j] = xs[j] > 0.5f * kNeg ? ex2f(xs[j] - m_run) : 0.f;
                l_run += (p[0] + p[1]) + (p[2] + p[3]);
                // weights as bf16 head + bf16 remainder
                const uint32_t ph0 = pack_bf16(p[0], p[1]), ph2 = pack_bf16(p[2], p[3]);
                const uint32_t pl0 = pack_bf16(p[0] - __uint_as_float(ph0 << 16), p[1] - __uint_as_float(ph0 & 0xffff0000u));
                const uint32_t pl2 = pack_bf16(p[2] - __uint_as_float(ph2 << 16), p[3] - __uint_as_float(ph2 & 0xffff0000u));
                // ---- acc += P V
#pragma unroll
                for (int t = 0; t < NT; t += 2) {
                    const int chunk = t + vc;
                    uint32_t vb[4];
                    ldsm_x4_t(vb, v_s + (chunk >> 3) * kDecBlock + vr * 128 + (((chunk & 7) ^ (vr & 7)) << 4));
                    mma_rows8(acc[t], ph0, ph2, vb[0], vb[1]);
                    mma_rows8(acc[t], pl0, pl2, vb[0], vb[1]);
                    mma_rows8(acc[t + 1], ph0, ph2, vb[2], vb[3]);
                    mma_rows8(acc[t + 1], pl0, pl2, vb[2], vb[3]);
                }
                if (row_w + 16 > rows) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar + 8 * s);
            }
            // row sum over the four lanes of a row; then this warp's (m, l, acc) to shared memory
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
            l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
            float* const mine = merge + (warp * 8 + g) * (D + 2);
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                mine[t * 8 + 2 * qd] = acc[t][0];
                mine[t * 8 + 2 * qd + 1] = acc[t][1];
            }
            if (qd == 0) { mine[D] = m_run; mine[D + 1] = l_run; }
            consumers_sync();
            const bool aborted = *abort_flag != 0;
            // merge the four warps (fixed order) and write this split's partial result
            if (!aborted) {
                float* const part = a.partial + (int64_t(x.u) * a.splits + x.sp) * a.group * (D + 2);
                for (int j = tid; j < a.group * (D + 2); j += 32 * kDecWarps) {
                    const int gg = j / (D + 2), c = j % (D + 2);
                    float m = kNeg;
#pragma unroll
                    for (int ww = 0; ww < kDecWarps; ++ww) m = fmaxf(m, merge[(ww * 8 + gg) * (D + 2) + D]);
                    float v = 0.f;
                    if (c == D) {
                        v = m;
                    } else {
#pragma unroll
                        for (int ww = 0; ww < kDecWarps; ++ww) {
                            const float* wm = merge + (ww * 8 + gg) * (D + 2);
                            v += wm[c] * ex2f(wm[D] - m);      // c == D + 1 sums the l's the same way
                        }
                    }
                    part[j] = v;
                }
            }
            // the barrier at the top of the next item also frees the merge area
        }
        if (*abort_flag && tid == 0) atomicOr(a.status, CSP_DEV_TIMEOUT);
    }
}

// out[b, hq, :] = sum_s acc_s 2^(m_s - m) / (n 2^-m + sum_s l_s 2^(m_s - m)) over the splits that had rows
__global__ void decode_merge_kernel(const DecodeArgs a) {
    const int u = blockIdx.x / a.group, g = blockIdx.x % a.group;
    const int b = u / a.n_kv_heads, h = u % a.n_kv_heads;
    const int D = a.head_dim;
    if (blockIdx.x == 0 && threadIdx.x == 0) *a.next_item = 0;     // the work counter is zero again for the next call
    int rows = a.n_rows[u];
    if ((rows < 0 || rows > a.capacity) && g == 0 && threadIdx.x == 0) atomicOr(a.status, CSP_DEV_BAD_LEN);
    rows = rows < 0 ? 0 : (rows > a.capacity ? a.capacity : rows);
    const int tiles = (rows + kDecTile - 1) / kDecTile;
    const int used = (tiles + a.tiles_per_split - 1) / a.tiles_per_split;
    float* const o = a.out + (int64_t(b) * a.n_kv_heads * a.group + h * a.group + g) * D;
    const float* const part = a.partial + (int64_t(u) * a.splits * a.group + g) * (D + 2);
    const int64_t stride = int64_t(a.group) * (D + 2);
    float m = kNeg;
    for (int s = 0; s < used; ++s) m = fmaxf(m, part[s * stride + D]);
    float l = 0.f;
    for (int s = 0; s < used; ++s) l += part[s * stride + D + 1] * ex2f(part[s * stride + D] - m);
    const float denom = a.n * ex2f(-m) + l;
    for (int c = threadIdx.x; c < D; c += blockDim.x) {
        float v = 0.f;
        for (int s = 0; s < used; ++s) v += part[s * stride + c] * ex2f(part[s * stride + D] - m);
        o[c] = (used > 0 && denom > 0.f) ? v / denom : 0.f;
    }
}

// csp_decode_step: the merge of decode_merge_kernel for all query heads of one unit, and then one query row of
// Eq. 1: the step's n-softmax weights, averaged over the query heads of the KV group, are added to the intra sum of
// the cached rows that carry the query's label and to the inter sum of the others.  On the first step of a window
// every slot of the unit is (over)written, so rows appended later start from zero.  One block per unit: the
// normalisers stay in shared memory, the logits are read once.
constexpr int kStepThreads = 256;
__global__ void __launch_bounds__(kStepThreads) decode_merge_accumulate_kernel(const DecodeArgs a) {
    __shared__ float ref[8], wgt[8];                 // per query head: reference exponent, 1 / (G (n 2^-m + l))
    const int u = blockIdx.x, b = u / a.n_kv_heads, h = u % a.n_kv_heads;
    const int D = a.head_dim, G = a.group;
    if (blockIdx.x == 0 && threadIdx.x == 0) *a.next_item = 0;     // the work counter is zero again for the next call
    int rows = a.n_rows[u];
    if ((rows < 0 || rows > a.capacity) && threadIdx.x == 0) atomicOr(a.status, CSP_DEV_BAD_LEN);
    rows = rows < 0 ? 0 : (rows > a.capacity ? a.capacity : rows);
    const int tiles = (rows + kDecTile - 1) / kDecTile;
    const int used = (tiles + a.tiles_per_split - 1) / a.tiles_per_split;
    const int64_t stride = int64_t(G) * (D + 2);
    for (int g = 0; g < G; ++g) {
        float* const o = a.out + (int64_t(b) * a.n_kv_heads * G + h * G + g) * D;
        const float* const part = a.partial + (int64_t(u) * a.splits * G + g) * (D + 2);
        float m = kNeg;
        for (int s = 0; s < used; ++s) m = fmaxf(m, part[s * stride + D]);
        float l = 0.f;
        for (int s = 0; s < used; ++s) l += part[s * stride + D + 1] * ex2f(part[s * stride + D] - m);
        const float denom = a.n * ex2f(-m) + l;
        const bool ok = used > 0 && denom > 0.f;
        if (threadIdx.x == 0) { ref[g] = m; wgt[g] = ok ? 1.0f / (float(G) * denom) : 0.f; }
        for (int c = threadIdx.x; c < D; c += kStepThreads) {
            float v = 0.f;
            for (int s = 0; s < used; ++s) v += part[s * stride + c] * ex2f(part[s * stride + D] - m);
            o[c] = ok ? v / denom : 0.f;
        }
    }
    __syncthreads();
    float* const as = a.acc_self + int64_t(u) * a.capacity;
    float* const ac = a.acc_cross + int64_t(u) * a.capacity;
    const uint8_t* const mod = a.modality + int64_t(b) * a.mod_sb + int64_t(h) * a.mod_sh;
    const uint32_t qlab = a.query_label[b];
    const float* const lg = a.logits + int64_t(u) * G * a.capacity;
    const int end = a.first_step ? a.capacity : rows;
    for (int t = threadIdx.x; t < end; t += kStepThreads) {
        if (t >= rows) { as[t] = 0.f; ac[t] = 0.f; continue; }
        float w = 0.f;
        for (int g = 0; g < G; ++g) w += ex2f(lg[int64_t(g) * a.capacity + t] - ref[g]) * wgt[g];
        const bool same = mod[t] == qlab;
        const float s0 = a.first_step ? 0.f : as[t], c0 = a.first_step ? 0.f : ac[t];
        as[t] = s0 + (same ? w : 0.f);
        ac[t] = c0 + (same ? 0.f : w);
    }
}

}  // namespace

int decode_splits(const csp_params& p) {
    const int units = p.batch * p.n_kv_heads;
    const int tiles = (p.out_capacity + kDecTile - 1) / kDecTile;
    if (units <= 0 || tiles <= 0) return 1;
    // at least about four work items per resident CTA (one per SM), but no item shorter than four tiles
    int splits = (4 * sm_count() + units - 1) / units;
    if (splits > (tiles + 3) / 4) splits = (tiles + 3) / 4;
    return splits < 1 ? 1 : splits;
}

size_t decode_workspace_bytes(const csp_params& p) {
    const size_t units = size_t(p.batch) * size_t(p.n_kv_heads);
    const size_t G = size_t(p.n_q_heads / p.n_kv_heads);
    return kStatusBytes + round256(units * size_t(decode_splits(p)) * G * size_t(p.head_dim + 2) * 4);
}

size_t decode_step_workspace_bytes(const csp_params& p) {
    const size_t units = size_t(p.batch) * size_t(p.n_kv_heads);
    const size_t G = size_t(p.n_q_heads / p.n_kv_heads);
    return decode_workspace_bytes(p) + round256(units * G * size_t(p.out_capacity) * 4);
}

csp_status launch_decode_attn(const csp_params& p, const csp_tensor& q, const csp_tensor& k, const csp_tensor& v,
                              const int32_t* n_rows, float* out, void* ws, cudaStream_t s, const DecodeStepArgs* step,
                              const csp_pages* pages) {
    if (p.dtype != CSP_BF16 || (p.head_dim != 64 && p.head_dim != 128)) return CSP_ERR_UNSUPPORTED;
    const int units = p.batch * p.n_kv_heads;
    if (units == 0) return CSP_OK;
    DecodeArgs a;
    a.logits = nullptr; a.modality = nullptr; a.mod_sb = a.mod_sh = 0; a.query_label = nullptr;
    a.acc_self = a.acc_cross = nullptr; a.first_step = 0;
    a.page_table = pages ? pages->page_table : nullptr;
    a.max_pages = pages ? pages->max_pages : 0;
    a.page_rows = pages ? pages->page_rows : 1;
    a.n_pages = pages ? pages->n_pages : 0;
    if (step) {
        a.logits = reinterpret_cast<float*>(static_cast<char*>(ws) + decode_workspace_bytes(p));
        a.modality = step->modality; a.mod_sb = step->mod_sb; a.mod_sh = step->mod_sh;
        a.query_label = step->query_label; a.acc_self = step->acc_self; a.acc_cross = step->acc_cross;
        a.first_step = step->first_step;
    }
    a.q = q.ptr; a.q_sb = q.stride_b; a.q_sh = q.stride_h;
    a.n_rows = n_rows;
    a.partial = reinterpret_cast<float*>(static_cast<char*>(ws) + kStatusBytes);
    a.out = out;
    a.status = static_cast<int32_t*>(ws);
    a.next_item = a.status + 8;
    a.n_kv_heads = p.n_kv_heads; a.group = p.n_q_heads / p.n_kv_heads; a.head_dim = p.head_dim;
    a.capacity = p.out_capacity;
    a.splits = decode_splits(p);
    const int tiles = (p.out_capacity + kDecTile - 1) / kDecTile;
    a.tiles_per_split = (tiles + a.splits - 1) / a.splits;
    a.n = p.n;
    a.scale_log2 = (p.scale > 0.f ? p.scale : 1.0f / sqrtf(float(p.head_dim))) * 1.4426950408889634f;
    if (p.out_capacity > 0) {
        CUtensorMap tk, tv;
        const int map_rows = pages ? pages->page_rows : p.out_capacity, map_outer = pages ? pages->n_pages : p.batch;
        if (!make_cache_tensor_map(&tk, k, p.dtype, p.head_dim, map_rows, p.n_kv_heads, map_outer, kDecTile) ||
            !make_cache_tensor_map(&tv, v, p.dtype, p.head_dim, map_rows, p.n_kv_heads, map_outer, kDecTile))
            return CSP_ERR_UNSUPPORTED;
        const int NH = p.head_dim / 64;
        const size_t smem = 1024 + size_t(kDecStages) * 2 * NH * kDecBlock + size_t(kDecWarps) * 8 * (p.head_dim + 2) * 4 +
                            16 * kDecStages + 64;
        auto kern = step ? (NH == 1 ? decode_attn_kernel<1, true> : decode_attn_kernel<2, true>)
                         : (NH == 1 ? decode_attn_kernel<1, false> : decode_attn_kernel<2, false>);
        static std::atomic<bool> configured[4][kMaxDevices];
        if (!raise_smem_limit(kern, int(smem), configured[(step ? 2 : 0) + NH - 1])) return CSP_ERR_CUDA;
        const int n_items = units * a.splits, sms = sm_count();
        kern<<<n_items < sms ? n_items : sms, kDecThreads, smem, s>>>(tk, tv, a, n_items);
        if (cudaGetLastError() != cudaSuccess) return CSP_ERR_CUDA;
    }
    if (step) decode_merge_accumulate_kernel<<<units, kStepThreads, 0, s>>>(a);
    else decode_merge_kernel<<<units * a.group, 128, 0, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? CSP_OK : CSP_ERR_CUDA;
}

}  // namespace csp
