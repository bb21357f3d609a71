// Internal declarations shared by the translation units of libcsp (not part of the C interface).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "csp.h"

namespace csp {

// ---- per-device host-side caches ----------------------------------------------------------
// Entry points may be called from several host threads at once.  What the launchers remember between
// calls (SM count, "this kernel's shared-memory limit has been raised on this device", how many clusters
// of a size fit on the device) sits in arrays of atomics indexed by the device ordinal: the cached values
// are the same whoever computes them, so a lost race only repeats an idempotent query.
constexpr int kMaxDevices = 64;
constexpr int kFallbackSms = 148;                    // B200; used only when the attribute query fails

// Streaming multiprocessors of the current device.
int sm_count();

// Raises a kernel's dynamic shared-memory limit the first time it is launched on the current device.
// `done` is that kernel's own array of per-device flags.
template <typename Kern>
inline bool raise_smem_limit(Kern kern, int bytes, std::atomic<bool> (&done)[kMaxDevices]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return false; }
    const bool cached = dev >= 0 && dev < kMaxDevices;
    if (cached && done[dev].load(std::memory_order_acquire)) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    if (cached) done[dev].store(true, std::memory_order_release);
    return true;
}

// ---- workspace layout -------------------------------------------------------------------
// [0, 256)            status area (word 0 = OR of CSP_DEV_* bits)
// then, each rounded up to 256 bytes:
//   score_self  fp32 [B, Hkv, max_len]     (prune_layer when the caller passes NULL)
//   score_cross fp32 [B, Hkv, max_len]
//   part_self   fp32 [B, Hkv, max_len]     (MEAN_ALL: per-KV-head partial sums)
//   part_cross  fp32 [B, Hkv, max_len]
//   keep_idx    int32 [B, Hkv, out_capacity]
//   order       int32 [B]                  (sequences by descending length, for load balance)
constexpr size_t kStatusBytes = 256;

struct WorkspaceLayout {
    size_t score_self, score_cross, part_self, part_cross, keep_idx, order, total;
};

inline size_t round256(size_t x) { return (x + 255) & ~size_t(255); }

inline WorkspaceLayout workspace_layout(const csp_params& p) {
    WorkspaceLayout w;
    const size_t units = size_t(p.batch) * size_t(p.n_kv_heads);
    const size_t sc = round256(units * size_t(p.max_len) * 4);
    w.score_self = kStatusBytes;
    w.score_cross = w.score_self + sc;
    w.part_self = w.score_cross + sc;
    w.part_cross = w.part_self + sc;
    w.keep_idx = w.part_cross + sc;
    w.order = w.keep_idx + round256(units * size_t(p.out_capacity) * 4);
    w.total = w.order + round256(size_t(p.batch) * 4);
    return w;
}

// ---- arguments handed to the kernels ------------------------------------------------------
struct ScoreArgs {
    const void* q; int64_t q_sb, q_sh, q_st;        // element strides
    const uint8_t* modality; int64_t mod_sb, mod_sh;
    const int32_t* seq_lens;
    const float* lse;                                // may be null
    float* score_self; float* score_cross;           // [B, Hkv, max_len]
    int32_t* status;
    int32_t* order_buf;                              // scratch for `order`, int32 [B]
    const int32_t* order;                            // null, or the sequences by descending length
    int32_t n_kv_heads, group, window, recent, max_len;
    float n, scale_log2, weight;                     // weight = 1/G or 1/Hq
    uint32_t* hist;                                  // null, or [B, Hkv, 2, CSP_HIST_BINS] counts to add to
    // paged cache: tile i of sequence b lies in page page_table[b * max_pages + i / tiles_per_page] of the pool,
    // at rows (i % tiles_per_page) * 128; null for a dense cache
    const int32_t* page_table; int32_t max_pages, tiles_per_page, n_pages;
};

// Coordinates of key tile `tile` of sequence `b` in the K tensor map: (first row, index on the outermost axis).
// Dense cache: (tile * 128, b).  Paged: a row inside the page that holds the tile, and that page.  A page
// number outside the pool gives an out-of-range coordinate: the copy then delivers zeros, it cannot fault; the
// call is flagged CSP_DEV_BAD_LEN.
__device__ __forceinline__ void tile_coords(const ScoreArgs& a, int tile, int b, int& row, int& outer) {
    if (a.page_table) {
        outer = a.page_table[int64_t(b) * a.max_pages + tile / a.tiles_per_page];
        row = (tile % a.tiles_per_page) * 128;
        if (outer < 0 || outer >= a.n_pages) { atomicOr(a.status, CSP_DEV_BAD_LEN); outer = a.n_pages; }
    } else {
        outer = b;
        row = tile * 128;
    }
}

struct SelectArgs {
    const float* score_self; const float* score_cross;
    const uint8_t* modality; int64_t mod_sb, mod_sh;
    const int32_t* seq_lens; const int32_t* budgets; const int32_t* total_budget;
    int32_t* keep_idx; int32_t* n_out; int32_t* status;
    int32_t n_kv_heads, window, recent, max_len, out_capacity;
    int32_t combine_and, global_mode;
    int32_t overall;                                 // global_mode with both problems on s + c and budgets [B, 1]
};

struct CompactArgs {
    const void* k; const void* v; void* k_out; void* v_out;
    int64_t k_sb, k_sh, k_st, v_sb, v_sh, v_st;      // in 16-byte units
    int64_t ko_sb, ko_sh, ko_st, vo_sb, vo_sh, vo_st;
    const uint8_t* modality; int64_t mod_sb, mod_sh; uint8_t* mod_out;
    const int32_t* keep_idx; const int32_t* n_out;
    int32_t n_kv_heads, max_len, out_capacity, chunks_per_row;
    int32_t* status;                                 // device status word, or null (csp_compact has none)
    // paged source (and, in place, destination): row t of sequence b lies in page page_table[b * max_pages +
    // t / page_rows] at row t % page_rows; k_sb / v_sb are then the page strides.  Null for a dense cache.
    const int32_t* page_table; int32_t max_pages, page_rows, n_pages;
};

// Cluster size (CTAs per unit, a power of two <= 8).  At least enough CTAs to occupy the `sms` SMs when
// there are few units; more when that lets every CTA keep all of its tiles' logits on chip
// (`tiles_kept` tiles per CTA; 0 if the kernel keeps none), which removes the second pass over K.
// Clusters of 4 and 8 fit on fewer SMs than single CTAs or pairs do (132 and 120 of a B200's 148), so when
// even 8 CTAs cannot keep the logits the cluster stays small: pairs, which also halves the longest CTA of
// a ragged batch.
inline int pick_cluster(int units, int max_tiles, int tiles_kept, int sms) {
    int c = 1;
    while (c < 8 && units * (c * 2) <= sms && c * 2 <= max_tiles) c *= 2;
    if (tiles_kept > 0 && (max_tiles + 7) / 8 <= tiles_kept) {
        while (c < 8 && (max_tiles + c - 1) / c > tiles_kept) c *= 2;
    } else if (tiles_kept > 0 && c < 2 && max_tiles >= 32) {
        c = 2;
    }
    return c;
}

// Host-visible checks of csp_prune_layer's arguments (everything but the workspace); enqueues nothing.
csp_status check_prune_layer_args(const csp_params* p, const csp_tensor& q_win, const csp_tensor& k, const csp_tensor& v,
                                  const uint8_t* modality, const int32_t* seq_lens, const int32_t* budgets,
                                  const csp_tensor& k_out, const csp_tensor& v_out, const int32_t* n_out);

// ---- host-side launchers (defined next to their kernels) ----------------------------------
csp_status launch_score(const csp_params& p, const ScoreArgs& a, const csp_tensor& k, cudaStream_t s,
                        const csp_pages* pages = nullptr);
csp_status launch_score_tc(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s);
csp_status launch_score_persist(const csp_params& p, const ScoreArgs& a, const CUtensorMap& tmap, cudaStream_t s,
                                bool* taken);
csp_status launch_ex2_probe(int fma_pipe, int iters, float* sink, size_t sink_elems, long long* n_exp, cudaStream_t s);
csp_status launch_hist_js(const csp_params& p, const uint32_t* hist, float* js, float* js_all, cudaStream_t s);
csp_status launch_head_mean(const csp_params& p, const float* part_self, const float* part_cross,
                            float* score_self, float* score_cross, const int32_t* seq_lens,
                            cudaStream_t s);
csp_status launch_select(const csp_params& p, const SelectArgs& a, cudaStream_t s);
constexpr int kSelectClusterMaxLen = 8 * 1024 * 8;   // longest cache the register-resident cluster select takes
csp_status launch_select_cluster(const csp_params& p, const SelectArgs& a, cudaStream_t s);
csp_status launch_compact(const csp_params& p, const CompactArgs& a, cudaStream_t s);
csp_status launch_select_compact(const csp_params& p, const SelectArgs& sa, const CompactArgs& ca, cudaStream_t s,
                                 bool* taken);

// 4-D tensor map over a cache [batch, heads, rows, head_dim] with 128-byte swizzle and boxes of 128 bytes x
// box_rows rows; false if the driver entry point is missing or the strides / alignment do not qualify.
bool make_cache_tensor_map(CUtensorMap* map, const csp_tensor& t, int dtype, int head_dim, int rows, int heads,
                           int batch, int box_rows);

// decode attention over the pruned cache (csp_decode.cu)
int decode_splits(const csp_params& p);
size_t decode_workspace_bytes(const csp_params& p);
// what csp_decode_step adds to a decode call: the labels and the running sums of Eq. 1
struct DecodeStepArgs {
    const uint8_t* modality; int64_t mod_sb, mod_sh;
    const uint8_t* query_label;
    float* acc_self; float* acc_cross;
    int32_t first_step;
};
size_t decode_step_workspace_bytes(const csp_params& p);
csp_status launch_decode_attn(const csp_params& p, const csp_tensor& q, const csp_tensor& k, const csp_tensor& v,
                              const int32_t* n_rows, float* out, void* ws, cudaStream_t s,
                              const DecodeStepArgs* step = nullptr, const csp_pages* pages = nullptr);

}  // namespace csp
