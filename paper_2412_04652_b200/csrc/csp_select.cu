// Selection kernel for caches longer than 65536 positions (shorter ones take csp_select_cluster.cu):
// the two top-K masks (Eq. 2), their combination (Eq. 3) and the ascending list
// of kept positions followed by the recent block (index side of Eq. 4).
//
// One CTA per (sequence, KV head) unit.  Up to four top-K problems run together (intra/inter score x
// text/visual keys, or intra/inter over all keys): an MSB-first radix select on the order-preserving
// integer image of the fp32 scores (staged once in shared memory) finds each problem's K-th value,
// ties at that value are taken in position order with a block-wide prefix count, and a second
// prefix count over the combined mask places the kept positions in ascending order.  The result equals the first K entries of a stable
// descending sort, exactly.
#include "csp_internal.cuh"

namespace csp {
namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kPasses = 3;                              // radix digits of 11, 11 and 10 bits
constexpr int kBins = 2048;
constexpr int kHistRow = kBins + kBins / 32;           // one pad word per 32 bins: conflict-free lane-strided scans
__device__ __forceinline__ int hpad(int bin) { return bin + (bin >> 5); }
constexpr int kBytesPerCached = 9;                      // two 32-bit keys and the label of one position
__device__ __constant__ int kDigitShift[kPasses] = {21, 10, 0};
__device__ __constant__ int kDigitBits[kPasses] = {11, 11, 10};

__device__ __forceinline__ uint32_t order_key(float f) {
    uint32_t b = __float_as_uint(f);
    if (b == 0x80000000u) b = 0u;                       // -0 ranks with +0
    return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u); // monotone: larger float <=> larger key
}

template <typename V>
__device__ __forceinline__ V block_exclusive_scan(V v, V* warp_tot, V* total_out) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    V inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const V o = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += o;
    }
    __syncthreads();                                    // warp_tot may still be read from a previous scan
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        V w = lane < kSelWarps ? warp_tot[lane] : V(0);
        V winc = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const V o = __shfl_up_sync(0xffffffffu, winc, d);
            if (lane >= d) winc += o;
        }
        warp_tot[lane] = winc - w;                      // exclusive prefix of the warp totals
        if (lane == 31) *total_out = winc;
    }
    __syncthreads();
    return warp_tot[warp] + inc - v;
}

__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(const SelectArgs a, const int n_cached_max) {
    // dynamic: hist[4][kBins], then the cached keys of the first n_cached positions
    extern __shared__ __align__(16) uint8_t sel_smem[];
    uint32_t (*hist)[kHistRow] = reinterpret_cast<uint32_t (*)[kHistRow]>(sel_smem);
    uint32_t* const cache_s = reinterpret_cast<uint32_t*>(sel_smem + 4 * kHistRow * 4);
    uint32_t* const cache_c = cache_s + n_cached_max;
    uint8_t* const cache_m = reinterpret_cast<uint8_t*>(cache_c + n_cached_max);
    __shared__ uint32_t prefix[4];
    __shared__ int32_t krem[4];
    __shared__ int32_t act[4];
    __shared__ unsigned long long scan_ws[kSelWarps];
    __shared__ unsigned long long scan_total[2];
    __shared__ uint32_t scan_ws32[kSelWarps];
    __shared__ uint32_t keep_total;

    const int u = blockIdx.x, b = u / a.n_kv_heads, h = u % a.n_kv_heads;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = a.seq_lens[b];
    int32_t* const idx = a.keep_idx + int64_t(u) * a.out_capacity;

    if (L < 0 || L > a.max_len) {
        if (tid == 0) { a.n_out[u] = -1; atomicOr(a.status, CSP_DEV_BAD_LEN); }
        return;
    }
    // Algorithm 1: a cache below its budget T (or too short for a window / recent block) is kept whole
    if (L < a.window || L < a.recent || (a.total_budget && L < a.total_budget[b])) {
        if (L > a.out_capacity) {
            if (tid == 0) { a.n_out[u] = -1; atomicOr(a.status, CSP_DEV_CAPACITY); }
            return;
        }
        for (int t = tid; t < L; t += kSelThreads) idx[t] = t;
        if (tid == 0) a.n_out[u] = L;
        return;
    }

    const int N = L - a.recent;
    const float* const ss = a.score_self + int64_t(u) * a.max_len;
    const float* const sc = a.score_cross + int64_t(u) * a.max_len;
    const uint8_t* const mod = a.modality + int64_t(b) * a.mod_sb + int64_t(h) * a.mod_sh;
    const int nprob = a.global_mode ? 2 : 4;
    const int32_t* const bud = a.budgets + int64_t(b) * (a.overall ? 1 : nprob);

    // stage the order-preserving keys and labels on chip once; every later pass reads them from there
    const int n_cached = min(N, n_cached_max);
    for (int t = tid; t < n_cached; t += kSelThreads) {
        cache_s[t] = order_key(a.overall ? ss[t] + sc[t] : ss[t]);
        cache_c[t] = order_key(a.overall ? ss[t] + sc[t] : sc[t]);
        cache_m[t] = mod[t];
    }
    auto key_s = [&](int t) { return t < n_cached ? cache_s[t] : order_key(a.overall ? ss[t] + sc[t] : ss[t]); };
    auto key_c = [&](int t) { return t < n_cached ? cache_c[t] : order_key(a.overall ? ss[t] + sc[t] : sc[t]); };
    auto label = [&](int t) { return t < n_cached ? cache_m[t] : mod[t]; };

    if (tid < 4) {
        prefix[tid] = 0;
        const int32_t k = tid < nprob ? bud[a.overall ? 0 : tid] : 0;
        krem[tid] = k;
        act[tid] = k > 0;
        if (k < 0) atomicOr(a.status, CSP_DEV_K_CLAMPED);
    }

    // ---- radix select, most significant digit first
    for (int pass = 0; pass < kPasses; ++pass) {
        const int shift = kDigitShift[pass], nbins = 1 << kDigitBits[pass];
        for (int i = tid; i < 4 * kHistRow; i += kSelThreads) (&hist[0][0])[i] = 0;
        __syncthreads();
        for (int t = tid; t < N; t += kSelThreads) {
            const int vis = a.global_mode ? 0 : (label(t) != 0);
            const int ps = vis, pc = a.global_mode ? 1 : 2 + vis;
            const uint32_t ks = key_s(t), kc = key_c(t);
            const uint32_t hi_s = pass == 0 ? 0u : ks >> (shift + kDigitBits[pass]);
            const uint32_t hi_c = pass == 0 ? 0u : kc >> (shift + kDigitBits[pass]);
            if (act[ps] && hi_s == prefix[ps]) atomicAdd(&hist[ps][hpad((ks >> shift) & (nbins - 1))], 1u);
            if (act[pc] && hi_c == prefix[pc]) atomicAdd(&hist[pc][hpad((kc >> shift) & (nbins - 1))], 1u);
        }
        __syncthreads();
        if (warp < nprob && act[warp]) {
            const int per_lane = nbins / 32;            // 64 or 32 bins per lane
            uint32_t ls = 0;
            for (int i = 0; i < per_lane; ++i) ls += hist[warp][hpad(lane * per_lane + i)];
            uint32_t suf = ls;                          // inclusive suffix sum over lanes
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_down_sync(0xffffffffu, suf, d);
                if (lane + d < 32) suf += o;
            }
            int32_t k = krem[warp];
            if (pass == 0) {
                const uint32_t total = __shfl_sync(0xffffffffu, suf, 0);   // candidates of this problem
                if (uint32_t(k) > total) {
                    k = int32_t(total);
                    if (lane == 0) atomicOr(a.status, CSP_DEV_K_CLAMPED);
                }
            }
            __syncwarp();
            if (k == 0) {
                if (lane == 0) { act[warp] = 0; krem[warp] = 0; }
            } else {
                const uint32_t above = suf - ls;
                if (above < uint32_t(k) && uint32_t(k) <= suf) {
                    uint32_t cum = above;
                    for (int i = per_lane - 1; i >= 0; --i) {
                        const uint32_t c = hist[warp][hpad(lane * per_lane + i)];
                        if (cum + c >= uint32_t(k)) {
                            prefix[warp] = (prefix[warp] << kDigitBits[pass]) | uint32_t(lane * per_lane + i);
                            krem[warp] = k - int32_t(cum);
                            break;
                        }
                        cum += c;
                    }
                }
            }
        }
        __syncthreads();
    }
    // now prefix[p] is the key of the K-th best of problem p and krem[p] how many keys equal to it are taken

    const int per = (N + kSelThreads - 1) / kSelThreads;
    const int t_beg = min(N, tid * per), t_end = min(N, t_beg + per);

    // ---- ties: rank of each threshold-valued key among its equals, in position order
    unsigned long long eq_self = 0, eq_cross = 0;       // two 32-bit counters each: [text | visual]
    for (int t = t_beg; t < t_end; ++t) {
        const int vis = a.global_mode ? 0 : (label(t) != 0);
        const int ps = vis, pc = a.global_mode ? 1 : 2 + vis;
        if (act[ps] && key_s(t) == prefix[ps]) eq_self += 1ull << (32 * vis);
        if (act[pc] && key_c(t) == prefix[pc]) eq_cross += 1ull << (32 * vis);
    }
    const unsigned long long ex_self = block_exclusive_scan(eq_self, scan_ws, &scan_total[0]);
    const unsigned long long ex_cross = block_exclusive_scan(eq_cross, scan_ws, &scan_total[1]);

    auto walk = [&](auto&& emit) {
        uint32_t rank_s[2] = {uint32_t(ex_self), uint32_t(ex_self >> 32)};
        uint32_t rank_c[2] = {uint32_t(ex_cross), uint32_t(ex_cross >> 32)};
        for (int t = t_beg; t < t_end; ++t) {
            const int vis = a.global_mode ? 0 : (label(t) != 0);
            const int ps = vis, pc = a.global_mode ? 1 : 2 + vis;
            const uint32_t ks = key_s(t), kc = key_c(t);
            bool sel_s = false, sel_c = false;
            if (act[ps]) {
                if (ks > prefix[ps]) sel_s = true;
                else if (ks == prefix[ps]) sel_s = int32_t(rank_s[vis]++) < krem[ps];
            }
            if (act[pc]) {
                if (kc > prefix[pc]) sel_c = true;
                else if (kc == prefix[pc]) sel_c = int32_t(rank_c[vis]++) < krem[pc];
            }
            emit(t, a.combine_and ? (sel_s && sel_c) : (sel_s || sel_c));   // Eq. 3
        }
    };

    uint32_t n_mine = 0;
    walk([&](int, bool keep) { n_mine += keep; });
    uint32_t pos = block_exclusive_scan(n_mine, scan_ws32, &keep_total);
    const int n_keep = int(keep_total);
    if (n_keep + a.recent > a.out_capacity) {
        if (tid == 0) { a.n_out[u] = -1; atomicOr(a.status, CSP_DEV_CAPACITY); }
        return;
    }
    walk([&](int t, bool keep) { if (keep) idx[pos++] = t; });
    for (int j = tid; j < a.recent; j += kSelThreads) idx[n_keep + j] = N + j;   // (+) the last R positions
    if (tid == 0) a.n_out[u] = n_keep + a.recent;
}

}  // namespace

csp_status launch_select(const csp_params& p, const SelectArgs& a, cudaStream_t s) {
    const int units = p.batch * p.n_kv_heads;
    if (units == 0) return CSP_OK;
    if (p.max_len <= kSelectClusterMaxLen) return launch_select_cluster(p, a, s);
    // very long caches: one CTA per unit, keys staged in shared memory as far as it reaches
    // cache as many positions on chip as one CTA's shared memory allows (the rest is read from L2)
    const size_t fixed = 4 * kHistRow * 4;
    size_t n_cached = size_t(p.max_len);
    const size_t limit = (200 * 1024 - fixed) / kBytesPerCached;
    if (n_cached > limit) n_cached = limit;
    n_cached = (n_cached + 3) & ~size_t(3);
    const size_t smem = fixed + n_cached * kBytesPerCached;
    static std::atomic<bool> configured[kMaxDevices];
    if (!raise_smem_limit(select_kernel, 227 * 1024 - 2048, configured)) return CSP_ERR_CUDA;
    select_kernel<<<units, kSelThreads, smem, s>>>(a, int(n_cached));
    return cudaGetLastError() == cudaSuccess ? CSP_OK : CSP_ERR_CUDA;
}

}  // namespace csp
