// Compaction kernel (Eq. 4): gather the kept rows of K and V, and their modality labels, into the
// compacted cache.  Pure data movement: rows are copied as 16-byte chunks, one row per
// (row bytes / 16) consecutive threads, so every load and store is a full 128-bit access and a
// warp covers whole rows.
#include "csp_internal.cuh"

namespace csp {
namespace {

constexpr int kCompactThreads = 256;
constexpr int kRowsPerCta = 64;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kCompactThreads) compact_kernel(const CompactArgs a) {
    const int blocks_per_unit = (a.out_capacity + kRowsPerCta - 1) / kRowsPerCta;
    const int u = blockIdx.x / blocks_per_unit, b = u / a.n_kv_heads, h = u % a.n_kv_heads;
    const int n = a.n_out[u];
    const int row0 = (blockIdx.x % blocks_per_unit) * kRowsPerCta;
    if (n <= 0 || row0 >= n) return;
    const int cpr = a.chunks_per_row;                    // 8, 16 or 32
    const int rows_per_iter = kCompactThreads / cpr;
    const int r_in = threadIdx.x / cpr, c = threadIdx.x % cpr;
    const int32_t* const idx = a.keep_idx + int64_t(u) * a.out_capacity;
    const uint4* const kin = static_cast<const uint4*>(a.k) + int64_t(b) * a.k_sb + int64_t(h) * a.k_sh;
    const uint4* const vin = static_cast<const uint4*>(a.v) + int64_t(b) * a.v_sb + int64_t(h) * a.v_sh;
    uint4* const kout = static_cast<uint4*>(a.k_out) + int64_t(b) * a.ko_sb + int64_t(h) * a.ko_sh;
    uint4* const vout = static_cast<uint4*>(a.v_out) + int64_t(b) * a.vo_sb + int64_t(h) * a.vo_sh;
    const int row_end = min(n, row0 + kRowsPerCta);

    for (int j0 = row0; j0 < row_end; j0 += 4 * rows_per_iter) {
        // four independent rows per thread in flight
        uint4 kv[4], vv[4];
        int jj[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            jj[q] = j0 + q * rows_per_iter + r_in;
            if (jj[q] < row_end) {
                const int t = idx[jj[q]];
                const bool ok = t >= 0 && t < a.max_len;   // a bad index copies nothing
                if (ok) {
                    kv[q] = ld_stream(kin + int64_t(t) * a.k_st + c);
                    vv[q] = ld_stream(vin + int64_t(t) * a.v_st + c);
                } else {
                    jj[q] = row_end;
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (jj[q] < row_end) {
                kout[int64_t(jj[q]) * a.ko_st + c] = kv[q];
                vout[int64_t(jj[q]) * a.vo_st + c] = vv[q];
            }
    }
    if (a.mod_out && a.modality) {
        const uint8_t* const mod = a.modality + int64_t(b) * a.mod_sb + int64_t(h) * a.mod_sh;
        for (int j = row0 + threadIdx.x; j < row_end; j += kCompactThreads) {
            const int t = idx[j];
            if (t >= 0 && t < a.max_len) a.mod_out[int64_t(u) * a.out_capacity + j] = mod[t];
        }
    }
}

}  // namespace

csp_status launch_compact(const csp_params& p, const CompactArgs& a, cudaStream_t s) {
    const int units = p.batch * p.n_kv_heads;
    if (units == 0 || p.out_capacity == 0) return CSP_OK;
    const long long blocks = (long long)((p.out_capacity + kRowsPerCta - 1) / kRowsPerCta) * units;
    if (blocks > 0x7fffffffLL) return CSP_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)blocks);
    compact_kernel<<<grid, kCompactThreads, 0, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? CSP_OK : CSP_ERR_CUDA;
}

}  // namespace csp
