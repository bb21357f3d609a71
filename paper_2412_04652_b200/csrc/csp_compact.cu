// Compaction kernels (Eq. 4): gather the kept rows of K and V, and their modality labels, into the
// compacted cache (a second buffer, or the same one: see compact_inplace_kernel).  Pure data movement: rows are copied as 16-byte chunks, one row per
// (row bytes / 16) consecutive threads, so every load and store is a full 128-bit access and a
// warp covers whole rows.
#include "csp_internal.cuh"

namespace csp {
namespace {

constexpr int kCompactThreads = 256;
// rows per CTA: 128 when that still gives every SM several CTAs (fewer, longer CTAs stream better), else 64
inline int rows_per_cta(int units, int capacity) {
    return (long long)units * ((capacity + 127) / 128) >= 8LL * sm_count() ? 128 : 64;
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Offset (in 16-byte units, before the chunk index) of row t of unit (b, h) in a source with strides (sb, sh, st):
// dense, or through the page table.  -1 for a row whose page number is outside the pool.
__device__ __forceinline__ int64_t row_offset(const CompactArgs& a, int b, int h, int t, int64_t sb, int64_t sh, int64_t st) {
    if (!a.page_table) return int64_t(b) * sb + int64_t(h) * sh + int64_t(t) * st;
    const int page = a.page_table[int64_t(b) * a.max_pages + t / a.page_rows];
    if (page < 0 || page >= a.n_pages) return -1;
    return int64_t(page) * sb + int64_t(h) * sh + int64_t(t % a.page_rows) * st;
}

template <int rows_cta, int CPR>   // rows per CTA; 16-byte chunks per row (8, 16 or 32)
__global__ void __launch_bounds__(kCompactThreads) compact_kernel(const CompactArgs a) {
    const int blocks_per_unit = (a.out_capacity + rows_cta - 1) / rows_cta;
    const int u = blockIdx.x / blocks_per_unit, b = u / a.n_kv_heads, h = u % a.n_kv_heads;
    int n = a.n_out[u];
    const int row0 = (blockIdx.x % blocks_per_unit) * rows_cta;
    if (n > a.out_capacity) {          // a row count the outputs cannot hold: copy what fits, say so where possible
        if (a.status && row0 == 0 && threadIdx.x == 0) atomicOr(a.status, CSP_DEV_CAPACITY);
        n = a.out_capacity;
    }
    if (n <= 0 || row0 >= n) return;
    constexpr int cpr = CPR;
    constexpr int rows_per_iter = kCompactThreads / cpr;
    const int r_in = threadIdx.x / cpr, c = threadIdx.x % cpr;
    const int32_t* const idx = a.keep_idx + int64_t(u) * a.out_capacity;
    const uint4* const kin = static_cast<const uint4*>(a.k);
    const uint4* const vin = static_cast<const uint4*>(a.v);
    uint4* const kout = static_cast<uint4*>(a.k_out) + int64_t(b) * a.ko_sb + int64_t(h) * a.ko_sh;
    uint4* const vout = static_cast<uint4*>(a.v_out) + int64_t(b) * a.vo_sb + int64_t(h) * a.vo_sh;
    const int row_end = min(n, row0 + rows_cta);

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
                const int64_t ko = ok ? row_offset(a, b, h, t, a.k_sb, a.k_sh, a.k_st) : -1;
                if (ko >= 0) {
                    kv[q] = ld_stream(kin + ko + c);
                    vv[q] = ld_stream(vin + row_offset(a, b, h, t, a.v_sb, a.v_sh, a.v_st) + c);
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

// In-place variant (k_out is k, v_out is v): row j of a unit moves from position keep_idx[j] >= j down to
// position j.  One CTA walks a unit's rows in ascending chunks; inside a chunk every load is issued before
// the CTA barrier and every store after it.  That is enough: a later chunk only reads positions at or beyond
// its own first row, which no earlier chunk has written, and a chunk's own sources are read before the
// barrier.  The loads are ordinary (coherent) loads: the kernel writes the memory it reads.
constexpr int kInplaceThreads = 512;

__global__ void __launch_bounds__(kInplaceThreads) compact_inplace_kernel(const CompactArgs a) {
    const int u = blockIdx.x, b = u / a.n_kv_heads, h = u % a.n_kv_heads;
    const int n = a.n_out[u];
    if (n <= 0) return;
    if (n > a.out_capacity && a.status && threadIdx.x == 0) atomicOr(a.status, CSP_DEV_CAPACITY);
    const int cpr = a.chunks_per_row;                    // 8, 16 or 32
    const int rows_per_iter = kInplaceThreads / cpr;
    const int r_in = threadIdx.x / cpr, c = threadIdx.x % cpr;
    const int32_t* const idx = a.keep_idx + int64_t(u) * a.out_capacity;
    uint4* const kio = static_cast<uint4*>(a.k_out);
    uint4* const vio = static_cast<uint4*>(a.v_out);
    const int row_end = min(n, a.out_capacity);
    // labels first: they go to a separate array, so no ordering is needed
    if (a.mod_out && a.modality) {
        const uint8_t* const mod = a.modality + int64_t(b) * a.mod_sb + int64_t(h) * a.mod_sh;
        for (int j = threadIdx.x; j < row_end; j += kInplaceThreads) {
            const int t = idx[j];
            if (t >= 0 && t < a.max_len) a.mod_out[int64_t(u) * a.out_capacity + j] = mod[t];
        }
    }
    for (int j0 = 0; j0 < row_end; j0 += 4 * rows_per_iter) {
        uint4 kv[4], vv[4];
        int jj[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            jj[q] = j0 + q * rows_per_iter + r_in;
            if (jj[q] < row_end) {
                const int t = idx[jj[q]];
                // a bad index or a source above its destination copies nothing; a row already in place stays
                const int64_t ko = (t > jj[q] && t < a.max_len) ? row_offset(a, b, h, t, a.ko_sb, a.ko_sh, a.ko_st) : -1;
                if (ko >= 0) {
                    kv[q] = kio[ko + c];
                    vv[q] = vio[row_offset(a, b, h, t, a.vo_sb, a.vo_sh, a.vo_st) + c];
                } else {
                    jj[q] = row_end;
                }
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (jj[q] < row_end) {
                const int64_t ko = row_offset(a, b, h, jj[q], a.ko_sb, a.ko_sh, a.ko_st);
                if (ko >= 0) {                       // the destination page of a kept row is one of the sequence's own
                    kio[ko + c] = kv[q];
                    vio[row_offset(a, b, h, jj[q], a.vo_sb, a.vo_sh, a.vo_st) + c] = vv[q];
                }
            }
    }
}

}  // namespace

csp_status launch_compact(const csp_params& p, const CompactArgs& a, cudaStream_t s) {
    const int units = p.batch * p.n_kv_heads;
    if (units == 0 || p.out_capacity == 0) return CSP_OK;
    if (a.k == a.k_out || a.v == a.v_out) {
        // in place: both tensors, with the strides of their inputs
        if (a.k != a.k_out || a.v != a.v_out || a.k_sb != a.ko_sb || a.k_sh != a.ko_sh || a.k_st != a.ko_st ||
            a.v_sb != a.vo_sb || a.v_sh != a.vo_sh || a.v_st != a.vo_st)
            return CSP_ERR_UNSUPPORTED;
        compact_inplace_kernel<<<units, kInplaceThreads, 0, s>>>(a);
        return cudaGetLastError() == cudaSuccess ? CSP_OK : CSP_ERR_CUDA;
    }
    const int rpc = rows_per_cta(units, p.out_capacity);
    const long long blocks = (long long)((p.out_capacity + rpc - 1) / rpc) * units;
    if (blocks > 0x7fffffffLL) return CSP_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)blocks);
    auto launch = [&](auto kern) { kern<<<grid, kCompactThreads, 0, s>>>(a); };
    switch (a.chunks_per_row) {
        case 8: rpc == 128 ? launch(compact_kernel<128, 8>) : launch(compact_kernel<64, 8>); break;
        case 16: rpc == 128 ? launch(compact_kernel<128, 16>) : launch(compact_kernel<64, 16>); break;
        case 32: rpc == 128 ? launch(compact_kernel<128, 32>) : launch(compact_kernel<64, 32>); break;
        default: return CSP_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? CSP_OK : CSP_ERR_CUDA;
}

}  // namespace csp
