// C interface of libcsp: argument checks, workspace carving and kernel sequencing.
#include <math.h>

#include "csp_internal.cuh"

namespace csp {
namespace {

csp_status check_arch() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CSP_ERR_CUDA; }
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return CSP_ERR_CUDA;
    }
    return major == 10 ? CSP_OK : CSP_ERR_ARCH;
}

int elem_size(const csp_params& p) { return p.dtype == CSP_F32 ? 4 : 2; }

csp_status check_params(const csp_params* p) {
    if (!p) return CSP_ERR_INVALID_ARG;
    if (p->batch < 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->head_dim <= 0 || p->window <= 0 ||
        p->recent < 0 || p->max_len < 0 || p->out_capacity < 0)
        return CSP_ERR_INVALID_ARG;
    if (p->dtype != CSP_F32 && p->dtype != CSP_BF16) return CSP_ERR_UNSUPPORTED;
    if (p->combine != CSP_COMBINE_OR && p->combine != CSP_COMBINE_AND) return CSP_ERR_INVALID_ARG;
    if (p->select_mode != CSP_SELECT_SEGMENTED && p->select_mode != CSP_SELECT_GLOBAL &&
        p->select_mode != CSP_SELECT_OVERALL)
        return CSP_ERR_INVALID_ARG;
    if (p->head_reduce != CSP_HEADS_PER_KV && p->head_reduce != CSP_HEADS_MEAN_ALL) return CSP_ERR_INVALID_ARG;
    if (p->n_q_heads % p->n_kv_heads) return CSP_ERR_INVALID_ARG;
    if (!(p->n >= 0.f) || !(p->scale >= 0.f)) return CSP_ERR_INVALID_ARG;
    const int row_bytes = p->head_dim * elem_size(*p);
    if (row_bytes != 128 && row_bytes != 256 && row_bytes != 512) return CSP_ERR_UNSUPPORTED;
    if (p->n_q_heads / p->n_kv_heads > 8) return CSP_ERR_UNSUPPORTED;
    if (p->window > 32) return CSP_ERR_UNSUPPORTED;
    // one (sequence, KV head) unit per grid row or plane: the product must fit a grid dimension
    if (int64_t(p->batch) * int64_t(p->n_kv_heads) > 65535) return CSP_ERR_UNSUPPORTED;
    return CSP_OK;
}

// base pointer and every stride must keep rows on 16-byte boundaries
bool tensor_ok(const csp_params& p, const csp_tensor& t) {
    const int64_t es = elem_size(p);
    return t.ptr && (uintptr_t(t.ptr) % 16 == 0) && (t.stride_b * es) % 16 == 0 && (t.stride_h * es) % 16 == 0 &&
           (t.stride_t * es) % 16 == 0 && t.stride_t >= 0 && t.stride_h >= 0 && t.stride_b >= 0;
}

csp_status check_workspace(const csp_params& p, void* ws, size_t bytes) {
    if (!ws || bytes < workspace_layout(p).total || (uintptr_t(ws) % 256)) return CSP_ERR_WORKSPACE;
    return CSP_OK;
}

csp_status do_score(const csp_params& p, const csp_tensor& q, const csp_tensor& k, const uint8_t* modality,
                    int64_t msb, int64_t msh, const int32_t* seq_lens, const float* lse, float* score_self,
                    float* score_cross, void* ws, cudaStream_t stream, uint32_t* hist = nullptr,
                    const csp_pages* pages = nullptr) {
    if (p.batch == 0 || p.max_len == 0) return CSP_OK;
    const WorkspaceLayout wl = workspace_layout(p);
    const bool mean_all = p.head_reduce == CSP_HEADS_MEAN_ALL && p.n_kv_heads > 1;
    if (p.head_reduce == CSP_HEADS_MEAN_ALL && msh != 0) return CSP_ERR_UNSUPPORTED;
    ScoreArgs a;
    a.q = q.ptr; a.q_sb = q.stride_b; a.q_sh = q.stride_h; a.q_st = q.stride_t;
    a.modality = modality; a.mod_sb = msb; a.mod_sh = msh;
    a.seq_lens = seq_lens; a.lse = lse;
    a.score_self = mean_all ? reinterpret_cast<float*>(static_cast<char*>(ws) + wl.part_self) : score_self;
    a.score_cross = mean_all ? reinterpret_cast<float*>(static_cast<char*>(ws) + wl.part_cross) : score_cross;
    a.status = static_cast<int32_t*>(ws);
    a.order_buf = reinterpret_cast<int32_t*>(static_cast<char*>(ws) + wl.order);
    a.order = nullptr;
    a.hist = hist;
    a.n_kv_heads = p.n_kv_heads; a.group = p.n_q_heads / p.n_kv_heads;
    a.window = p.window; a.recent = p.recent; a.max_len = p.max_len;
    a.n = p.n;
    const float scale = p.scale > 0.f ? p.scale : 1.0f / sqrtf(float(p.head_dim));
    a.scale_log2 = scale * 1.4426950408889634f;
    a.weight = p.head_reduce == CSP_HEADS_MEAN_ALL ? 1.0f / float(p.n_q_heads) : 1.0f / float(a.group);
    csp_status st = launch_score(p, a, k, stream, pages);
    if (st != CSP_OK) return st;
    if (mean_all) st = launch_head_mean(p, a.score_self, a.score_cross, score_self, score_cross, seq_lens, stream);
    return st;
}

SelectArgs select_args(const csp_params& p, const float* score_self, const float* score_cross,
                       const uint8_t* modality, int64_t msb, int64_t msh, const int32_t* seq_lens,
                       const int32_t* budgets, const int32_t* total_budget, int32_t* keep_idx, int32_t* n_out,
                       void* ws) {
    SelectArgs a;
    a.score_self = score_self; a.score_cross = score_cross;
    a.modality = modality; a.mod_sb = msb; a.mod_sh = msh;
    a.seq_lens = seq_lens; a.budgets = budgets; a.total_budget = total_budget;
    a.keep_idx = keep_idx; a.n_out = n_out; a.status = static_cast<int32_t*>(ws);
    a.n_kv_heads = p.n_kv_heads; a.window = p.window; a.recent = p.recent; a.max_len = p.max_len;
    a.out_capacity = p.out_capacity;
    a.combine_and = p.combine == CSP_COMBINE_AND;
    // OVERALL runs as GLOBAL with both problems on the summed score and the same budget: their union is the one top-K
    a.overall = p.select_mode == CSP_SELECT_OVERALL;
    a.global_mode = p.select_mode == CSP_SELECT_GLOBAL || a.overall;
    return a;
}

csp_status do_select(const csp_params& p, const float* score_self, const float* score_cross,
                     const uint8_t* modality, int64_t msb, int64_t msh, const int32_t* seq_lens,
                     const int32_t* budgets, const int32_t* total_budget, int32_t* keep_idx, int32_t* n_out,
                     void* ws, cudaStream_t stream) {
    return launch_select(p, select_args(p, score_self, score_cross, modality, msb, msh, seq_lens, budgets, total_budget,
                                        keep_idx, n_out, ws), stream);
}

CompactArgs compact_args(const csp_params& p, const csp_tensor& k, const csp_tensor& v, const uint8_t* modality,
                         int64_t msb, int64_t msh, const int32_t* keep_idx, const int32_t* n_out,
                         const csp_tensor& k_out, const csp_tensor& v_out, uint8_t* mod_out, int32_t* status,
                         const csp_pages* pages) {
    const int64_t es = elem_size(p);
    CompactArgs a;
    a.k = k.ptr; a.v = v.ptr; a.k_out = k_out.ptr; a.v_out = v_out.ptr;
    a.k_sb = k.stride_b * es / 16; a.k_sh = k.stride_h * es / 16; a.k_st = k.stride_t * es / 16;
    a.v_sb = v.stride_b * es / 16; a.v_sh = v.stride_h * es / 16; a.v_st = v.stride_t * es / 16;
    a.ko_sb = k_out.stride_b * es / 16; a.ko_sh = k_out.stride_h * es / 16; a.ko_st = k_out.stride_t * es / 16;
    a.vo_sb = v_out.stride_b * es / 16; a.vo_sh = v_out.stride_h * es / 16; a.vo_st = v_out.stride_t * es / 16;
    a.modality = modality; a.mod_sb = msb; a.mod_sh = msh; a.mod_out = mod_out;
    a.keep_idx = keep_idx; a.n_out = n_out;
    a.n_kv_heads = p.n_kv_heads; a.max_len = p.max_len; a.out_capacity = p.out_capacity;
    a.chunks_per_row = int(p.head_dim * es / 16);
    a.status = status;
    a.page_table = pages ? pages->page_table : nullptr;
    a.max_pages = pages ? pages->max_pages : 0;
    a.page_rows = pages ? pages->page_rows : 1;
    a.n_pages = pages ? pages->n_pages : 0;
    return a;
}

csp_status do_compact(const csp_params& p, const csp_tensor& k, const csp_tensor& v, const uint8_t* modality,
                      int64_t msb, int64_t msh, const int32_t* keep_idx, const int32_t* n_out,
                      const csp_tensor& k_out, const csp_tensor& v_out, uint8_t* mod_out, int32_t* status,
                      cudaStream_t stream, const csp_pages* pages = nullptr) {
    return launch_compact(p, compact_args(p, k, v, modality, msb, msh, keep_idx, n_out, k_out, v_out, mod_out, status,
                                          pages), stream);
}

// Selection and compaction of one call: the fused persistent kernel where the shape qualifies (many units whose
// selection fits one CTA, dense second output buffers), else the two kernels one after the other.
csp_status do_select_compact(const csp_params& p, const float* ss, const float* sc, const csp_tensor& k,
                             const csp_tensor& v, const uint8_t* modality, int64_t msb, int64_t msh,
                             const int32_t* seq_lens, const int32_t* budgets, const int32_t* total_budget,
                             int32_t* idx, int32_t* n_out, const csp_tensor& k_out, const csp_tensor& v_out,
                             uint8_t* mod_out, void* ws, cudaStream_t stream, bool allow_fused) {
    const SelectArgs sa = select_args(p, ss, sc, modality, msb, msh, seq_lens, budgets, total_budget, idx, n_out, ws);
    const CompactArgs ca = compact_args(p, k, v, modality, msb, msh, idx, n_out, k_out, v_out, mod_out,
                                        static_cast<int32_t*>(ws), nullptr);
    if (allow_fused) {
        bool taken = false;
        const csp_status st = launch_select_compact(p, sa, ca, stream, &taken);
        if (st != CSP_OK || taken) return st;
    }
    const csp_status st = launch_select(p, sa, stream);
    return st != CSP_OK ? st : launch_compact(p, ca, stream);
}

}  // namespace

int sm_count() {
    static std::atomic<int> cache[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return kFallbackSms; }
    const bool cached = dev >= 0 && dev < kMaxDevices;
    if (cached) {
        const int v = cache[dev].load(std::memory_order_relaxed);
        if (v > 0) return v;
    }
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return kFallbackSms;
    }
    if (cached) cache[dev].store(n, std::memory_order_relaxed);
    return n;
}

csp_status check_prune_layer_args(const csp_params* p, const csp_tensor& q_win, const csp_tensor& k, const csp_tensor& v,
                                  const uint8_t* modality, const int32_t* seq_lens, const int32_t* budgets,
                                  const csp_tensor& k_out, const csp_tensor& v_out, const int32_t* n_out) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!modality || !seq_lens || !budgets || !n_out || !q_win.ptr || !k.ptr || !v.ptr || !k_out.ptr || !v_out.ptr)
        return CSP_ERR_INVALID_ARG;
    if (!tensor_ok(*p, q_win) || !tensor_ok(*p, k) || !tensor_ok(*p, v) || !tensor_ok(*p, k_out) ||
        !tensor_ok(*p, v_out))
        return CSP_ERR_UNSUPPORTED;
    return check_arch();
}

namespace {
// csp_prune_layer; `v_on_device` is false when V is page-locked host memory read over the bus, which keeps the
// compaction kernel with many small CTAs (more requests in flight than one resident CTA per SM has)
csp_status prune_layer_impl(const csp_params* p, const csp_tensor& q_win, const csp_tensor& k, const csp_tensor& v,
                            const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                            const int32_t* seq_lens, const int32_t* budgets, const int32_t* total_budget_or_null,
                            const float* lse_or_null, const csp_tensor& k_out, const csp_tensor& v_out, uint8_t* mod_out,
                            int32_t* n_out, float* score_self_or_null, float* score_cross_or_null,
                            int32_t* keep_idx_or_null, void* workspace, size_t workspace_bytes, void* cuda_stream,
                            bool v_on_device) {
    csp_status st = check_prune_layer_args(p, q_win, k, v, modality, seq_lens, budgets, k_out, v_out, n_out);
    if (st != CSP_OK) return st;
    if ((st = check_workspace(*p, workspace, workspace_bytes)) != CSP_OK) return st;
    const WorkspaceLayout wl = workspace_layout(*p);
    char* ws = static_cast<char*>(workspace);
    float* ss = score_self_or_null ? score_self_or_null : reinterpret_cast<float*>(ws + wl.score_self);
    float* sc = score_cross_or_null ? score_cross_or_null : reinterpret_cast<float*>(ws + wl.score_cross);
    int32_t* idx = keep_idx_or_null ? keep_idx_or_null : reinterpret_cast<int32_t*>(ws + wl.keep_idx);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if ((st = do_score(*p, q_win, k, modality, mod_stride_b, mod_stride_h, seq_lens, lse_or_null, ss, sc,
                       workspace, stream)) != CSP_OK)
        return st;
    return do_select_compact(*p, ss, sc, k, v, modality, mod_stride_b, mod_stride_h, seq_lens, budgets,
                             total_budget_or_null, idx, n_out, k_out, v_out, mod_out, workspace, stream, v_on_device);
}

}  // namespace

}  // namespace csp

using namespace csp;

extern "C" {

size_t csp_workspace_bytes(const csp_params* p) {
    if (check_params(p) != CSP_OK) return 0;
    return workspace_layout(*p).total;
}

csp_status csp_workspace_reset(void* workspace, void* cuda_stream) {
    if (!workspace) return CSP_ERR_WORKSPACE;
    if (cudaMemsetAsync(workspace, 0, kStatusBytes, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        cudaGetLastError();
        return CSP_ERR_CUDA;
    }
    return CSP_OK;
}

csp_status csp_score(const csp_params* p, csp_tensor q_win, csp_tensor k, const uint8_t* modality,
                     int64_t mod_stride_b, int64_t mod_stride_h, const int32_t* seq_lens,
                     const float* lse_or_null, float* score_self, float* score_cross, void* workspace,
                     size_t workspace_bytes, void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!modality || !seq_lens || !score_self || !score_cross || !q_win.ptr || !k.ptr) return CSP_ERR_INVALID_ARG;
    if (!tensor_ok(*p, q_win) || !tensor_ok(*p, k)) return CSP_ERR_UNSUPPORTED;
    if ((st = check_workspace(*p, workspace, workspace_bytes)) != CSP_OK) return st;
    if ((st = check_arch()) != CSP_OK) return st;
    return do_score(*p, q_win, k, modality, mod_stride_b, mod_stride_h, seq_lens, lse_or_null, score_self,
                    score_cross, workspace, static_cast<cudaStream_t>(cuda_stream));
}

csp_status csp_select(const csp_params* p, const float* score_self, const float* score_cross,
                      const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                      const int32_t* seq_lens, const int32_t* budgets, const int32_t* total_budget_or_null,
                      int32_t* keep_idx, int32_t* n_out, void* workspace, size_t workspace_bytes,
                      void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!score_self || !score_cross || !modality || !seq_lens || !budgets || !keep_idx || !n_out)
        return CSP_ERR_INVALID_ARG;
    if ((st = check_workspace(*p, workspace, workspace_bytes)) != CSP_OK) return st;
    if ((st = check_arch()) != CSP_OK) return st;
    return do_select(*p, score_self, score_cross, modality, mod_stride_b, mod_stride_h, seq_lens, budgets,
                     total_budget_or_null, keep_idx, n_out, workspace, static_cast<cudaStream_t>(cuda_stream));
}

csp_status csp_compact(const csp_params* p, csp_tensor k, csp_tensor v, const uint8_t* modality,
                       int64_t mod_stride_b, int64_t mod_stride_h, const int32_t* keep_idx, const int32_t* n_out,
                       csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out, void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!keep_idx || !n_out || !k.ptr || !v.ptr || !k_out.ptr || !v_out.ptr) return CSP_ERR_INVALID_ARG;
    if (mod_out && !modality) return CSP_ERR_INVALID_ARG;
    if (!tensor_ok(*p, k) || !tensor_ok(*p, v) || !tensor_ok(*p, k_out) || !tensor_ok(*p, v_out))
        return CSP_ERR_UNSUPPORTED;
    if ((st = check_arch()) != CSP_OK) return st;
    return do_compact(*p, k, v, modality, mod_stride_b, mod_stride_h, keep_idx, n_out, k_out, v_out, mod_out,
                      nullptr, static_cast<cudaStream_t>(cuda_stream));
}

csp_status csp_select_compact(const csp_params* p, const float* score_self, const float* score_cross, csp_tensor k,
                              csp_tensor v, const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                              const int32_t* seq_lens, const int32_t* budgets, const int32_t* total_budget_or_null,
                              csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out, int32_t* n_out,
                              int32_t* keep_idx_or_null, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!score_self || !score_cross || !modality || !seq_lens || !budgets || !n_out || !k.ptr || !v.ptr || !k_out.ptr ||
        !v_out.ptr)
        return CSP_ERR_INVALID_ARG;
    if (!tensor_ok(*p, k) || !tensor_ok(*p, v) || !tensor_ok(*p, k_out) || !tensor_ok(*p, v_out)) return CSP_ERR_UNSUPPORTED;
    if ((st = check_workspace(*p, workspace, workspace_bytes)) != CSP_OK) return st;
    if ((st = check_arch()) != CSP_OK) return st;
    int32_t* idx = keep_idx_or_null ? keep_idx_or_null
                                    : reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + workspace_layout(*p).keep_idx);
    return do_select_compact(*p, score_self, score_cross, k, v, modality, mod_stride_b, mod_stride_h, seq_lens, budgets,
                             total_budget_or_null, idx, n_out, k_out, v_out, mod_out, workspace,
                             static_cast<cudaStream_t>(cuda_stream), true);
}

csp_status csp_prune_layer(const csp_params* p, csp_tensor q_win, csp_tensor k, csp_tensor v,
                           const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                           const int32_t* seq_lens, const int32_t* budgets, const int32_t* total_budget_or_null,
                           const float* lse_or_null, csp_tensor k_out, csp_tensor v_out, uint8_t* mod_out,
                           int32_t* n_out, float* score_self_or_null, float* score_cross_or_null,
                           int32_t* keep_idx_or_null, void* workspace, size_t workspace_bytes,
                           void* cuda_stream) {
    return prune_layer_impl(p, q_win, k, v, modality, mod_stride_b, mod_stride_h, seq_lens, budgets,
                            total_budget_or_null, lse_or_null, k_out, v_out, mod_out, n_out, score_self_or_null,
                            score_cross_or_null, keep_idx_or_null, workspace, workspace_bytes, cuda_stream, true);
}

// A page table must cover max_len positions with pages of whole 128-key tiles.
static csp_status check_pages(const csp_params& p, const csp_pages* pg) {
    if (!pg || !pg->page_table) return CSP_ERR_INVALID_ARG;
    if (pg->page_rows <= 0 || pg->page_rows % 128 || pg->max_pages <= 0 || pg->n_pages <= 0) return CSP_ERR_INVALID_ARG;
    if (int64_t(pg->max_pages) * pg->page_rows < p.max_len) return CSP_ERR_INVALID_ARG;
    if (p.dtype != CSP_BF16 || p.head_reduce != CSP_HEADS_PER_KV) return CSP_ERR_UNSUPPORTED;
    return CSP_OK;
}

csp_status csp_prune_layer_paged(const csp_params* p, csp_tensor q_win, csp_tensor k_pool, csp_tensor v_pool,
                                 const csp_pages* pages, const uint8_t* modality, int64_t mod_stride_b,
                                 int64_t mod_stride_h, const int32_t* seq_lens, const int32_t* budgets,
                                 const int32_t* total_budget_or_null, const float* lse_or_null, csp_tensor k_out,
                                 csp_tensor v_out, uint8_t* mod_out, int32_t* n_out, float* score_self_or_null,
                                 float* score_cross_or_null, int32_t* keep_idx_or_null, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
    csp_status st = check_prune_layer_args(p, q_win, k_pool, v_pool, modality, seq_lens, budgets, k_out, v_out, n_out);
    if (st != CSP_OK) return st;
    if ((st = check_pages(*p, pages)) != CSP_OK) return st;
    // in place, the kept rows are addressed through the table as well: it must cover the output capacity
    if (k_out.ptr == k_pool.ptr && int64_t(pages->max_pages) * pages->page_rows < p->out_capacity) return CSP_ERR_INVALID_ARG;
    if ((st = check_workspace(*p, workspace, workspace_bytes)) != CSP_OK) return st;
    const WorkspaceLayout wl = workspace_layout(*p);
    char* ws = static_cast<char*>(workspace);
    float* ss = score_self_or_null ? score_self_or_null : reinterpret_cast<float*>(ws + wl.score_self);
    float* sc = score_cross_or_null ? score_cross_or_null : reinterpret_cast<float*>(ws + wl.score_cross);
    int32_t* idx = keep_idx_or_null ? keep_idx_or_null : reinterpret_cast<int32_t*>(ws + wl.keep_idx);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if ((st = do_score(*p, q_win, k_pool, modality, mod_stride_b, mod_stride_h, seq_lens, lse_or_null, ss, sc,
                       workspace, stream, nullptr, pages)) != CSP_OK)
        return st;
    if ((st = do_select(*p, ss, sc, modality, mod_stride_b, mod_stride_h, seq_lens, budgets, total_budget_or_null,
                        idx, n_out, workspace, stream)) != CSP_OK)
        return st;
    return do_compact(*p, k_pool, v_pool, modality, mod_stride_b, mod_stride_h, idx, n_out, k_out, v_out, mod_out,
                      static_cast<int32_t*>(workspace), stream, pages);
}

// staging layout for the host-buffer variant: every block rounded up to 256 bytes
namespace {
struct StagingLayout {
    size_t q, k, v, mod, seq, bud, tot, k_out, v_out, mod_out, n_out, ws, total;
};
StagingLayout staging_layout(const csp_params& p, int mod_per_head) {
    StagingLayout s;
    const size_t es = size_t(elem_size(p)), units = size_t(p.batch) * p.n_kv_heads;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += round256(bytes); return o; };
    s.q = take(size_t(p.batch) * p.n_q_heads * p.window * p.head_dim * es);
    s.k = take(units * p.max_len * p.head_dim * es);
    s.v = take(units * p.max_len * p.head_dim * es);
    s.mod = take((mod_per_head ? units : size_t(p.batch)) * p.max_len);
    s.seq = take(size_t(p.batch) * 4);
    s.bud = take(size_t(p.batch) * 16);
    s.tot = take(size_t(p.batch) * 4);
    s.k_out = take(units * p.out_capacity * p.head_dim * es);
    s.v_out = take(units * p.out_capacity * p.head_dim * es);
    s.mod_out = take(units * p.out_capacity);
    s.n_out = take(units * 4);
    s.ws = take(workspace_layout(p).total);
    s.total = off;
    return s;
}
}  // namespace

size_t csp_host_staging_bytes(const csp_params* p) {
    if (check_params(p) != CSP_OK) return 0;
    return staging_layout(*p, 1).total;
}

csp_status csp_prune_layer_host(const csp_params* p, const void* q_host, const void* k_host, const void* v_host,
                                const uint8_t* modality_host, int mod_per_head, const int32_t* seq_lens_host,
                                const int32_t* budgets_host, const int32_t* total_budget_host_or_null,
                                void* k_out_host, void* v_out_host, uint8_t* mod_out_host, int32_t* n_out_host,
                                int32_t* dev_status_host, void* staging, size_t staging_bytes, void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!q_host || !k_host || !v_host || !modality_host || !seq_lens_host || !budgets_host || !k_out_host ||
        !v_out_host || !n_out_host)
        return CSP_ERR_INVALID_ARG;
    const StagingLayout sl = staging_layout(*p, mod_per_head ? 1 : 0);
    if (!staging || staging_bytes < sl.total || (uintptr_t(staging) % 256)) return CSP_ERR_WORKSPACE;
    if ((st = check_arch()) != CSP_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char* d = static_cast<char*>(staging);
    const size_t es = size_t(elem_size(*p)), units = size_t(p->batch) * p->n_kv_heads;
    const size_t q_bytes = size_t(p->batch) * p->n_q_heads * p->window * p->head_dim * es;
    const size_t kv_bytes = units * p->max_len * p->head_dim * es;
    const size_t mod_bytes = (mod_per_head ? units : size_t(p->batch)) * p->max_len;
    const size_t out_bytes = units * p->out_capacity * p->head_dim * es;
    const int nbud = p->select_mode == CSP_SELECT_GLOBAL ? 2 : (p->select_mode == CSP_SELECT_OVERALL ? 1 : 4);
    bool ok = true;
    auto h2d = [&](size_t off, const void* src, size_t bytes) {
        if (bytes) ok = ok && cudaMemcpyAsync(d + off, src, bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    };
    auto d2h = [&](void* dst, size_t off, size_t bytes) {
        if (bytes) ok = ok && cudaMemcpyAsync(dst, d + off, bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    };
    // V is only ever read at the kept rows.  When the caller's buffer is page-locked memory that this device can
    // address (cudaHostAlloc / cudaHostRegister), the compaction kernel fetches those rows from it directly and
    // the copy of the whole tensor is skipped; pageable or misaligned memory is staged in full as before.
    const void* v_mapped = nullptr;
    {
        cudaPointerAttributes at;
        int can_map = 0, dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&can_map, cudaDevAttrCanMapHostMemory, dev) == cudaSuccess && can_map &&
            cudaPointerGetAttributes(&at, v_host) == cudaSuccess && at.type == cudaMemoryTypeHost &&
            at.devicePointer && (uintptr_t(at.devicePointer) % 16 == 0))
            v_mapped = at.devicePointer;
        cudaGetLastError();
    }
    h2d(sl.q, q_host, q_bytes);
    h2d(sl.k, k_host, kv_bytes);
    if (!v_mapped) h2d(sl.v, v_host, kv_bytes);
    h2d(sl.mod, modality_host, mod_bytes);
    h2d(sl.seq, seq_lens_host, size_t(p->batch) * 4);
    h2d(sl.bud, budgets_host, size_t(p->batch) * 4 * nbud);
    if (total_budget_host_or_null) h2d(sl.tot, total_budget_host_or_null, size_t(p->batch) * 4);
    ok = ok && cudaMemsetAsync(d + sl.ws, 0, kStatusBytes, stream) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return CSP_ERR_CUDA; }

    const int64_t d_ = p->head_dim;
    csp_tensor q = {d + sl.q, int64_t(p->n_q_heads) * p->window * d_, int64_t(p->window) * d_, d_};
    csp_tensor k = {d + sl.k, int64_t(p->n_kv_heads) * p->max_len * d_, int64_t(p->max_len) * d_, d_};
    csp_tensor v = {v_mapped ? const_cast<void*>(v_mapped) : static_cast<void*>(d + sl.v), k.stride_b, k.stride_h, d_};
    csp_tensor ko = {d + sl.k_out, int64_t(p->n_kv_heads) * p->out_capacity * d_, int64_t(p->out_capacity) * d_, d_};
    csp_tensor vo = {d + sl.v_out, ko.stride_b, ko.stride_h, d_};
    const int64_t msb = mod_per_head ? int64_t(p->n_kv_heads) * p->max_len : p->max_len;
    const int64_t msh = mod_per_head ? p->max_len : 0;
    st = prune_layer_impl(p, q, k, v, reinterpret_cast<uint8_t*>(d + sl.mod), msb, msh,
                          reinterpret_cast<int32_t*>(d + sl.seq), reinterpret_cast<int32_t*>(d + sl.bud),
                          total_budget_host_or_null ? reinterpret_cast<int32_t*>(d + sl.tot) : nullptr, nullptr, ko, vo,
                          reinterpret_cast<uint8_t*>(d + sl.mod_out), reinterpret_cast<int32_t*>(d + sl.n_out),
                          nullptr, nullptr, nullptr, d + sl.ws, workspace_layout(*p).total, cuda_stream,
                          v_mapped == nullptr);
    if (st != CSP_OK) return st;
    d2h(k_out_host, sl.k_out, out_bytes);
    d2h(v_out_host, sl.v_out, out_bytes);
    if (mod_out_host) d2h(mod_out_host, sl.mod_out, units * p->out_capacity);
    d2h(n_out_host, sl.n_out, units * 4);
    if (dev_status_host) d2h(dev_status_host, sl.ws, 4);
    ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return CSP_ERR_CUDA; }
    return CSP_OK;
}

size_t csp_decode_workspace_bytes(const csp_params* p) {
    if (check_params(p) != CSP_OK) return 0;
    return decode_workspace_bytes(*p);
}

csp_status csp_decode_attn(const csp_params* p, csp_tensor q, csp_tensor k, csp_tensor v, const int32_t* n_rows,
                           float* out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!q.ptr || !k.ptr || !v.ptr || !n_rows || !out) return CSP_ERR_INVALID_ARG;
    if (p->dtype != CSP_BF16 || (p->head_dim != 64 && p->head_dim != 128)) return CSP_ERR_UNSUPPORTED;
    if (!tensor_ok(*p, q) || !tensor_ok(*p, k) || !tensor_ok(*p, v)) return CSP_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < decode_workspace_bytes(*p) || (uintptr_t(workspace) % 256))
        return CSP_ERR_WORKSPACE;
    if ((st = check_arch()) != CSP_OK) return st;
    return launch_decode_attn(*p, q, k, v, n_rows, out, workspace, static_cast<cudaStream_t>(cuda_stream));
}

csp_status csp_weight_histogram(const csp_params* p, csp_tensor q_win, csp_tensor k, const uint8_t* modality,
                                int64_t mod_stride_b, int64_t mod_stride_h, const int32_t* seq_lens,
                                const float* lse_or_null, uint32_t* hist, float* js_or_null, float* js_all_or_null,
                                void* workspace, size_t workspace_bytes, void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!modality || !seq_lens || !hist || !q_win.ptr || !k.ptr) return CSP_ERR_INVALID_ARG;
    if (p->dtype != CSP_BF16 || p->head_reduce != CSP_HEADS_PER_KV) return CSP_ERR_UNSUPPORTED;
    if (!tensor_ok(*p, q_win) || !tensor_ok(*p, k)) return CSP_ERR_UNSUPPORTED;
    if ((st = check_workspace(*p, workspace, workspace_bytes)) != CSP_OK) return st;
    if ((st = check_arch()) != CSP_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t units = size_t(p->batch) * p->n_kv_heads;
    if (units == 0) return CSP_OK;
    if (cudaMemsetAsync(hist, 0, units * 2 * CSP_HIST_BINS * sizeof(uint32_t), stream) != cudaSuccess) {
        cudaGetLastError();
        return CSP_ERR_CUDA;
    }
    // the scores themselves are a by-product here: they land in the workspace
    const WorkspaceLayout wl = workspace_layout(*p);
    char* ws = static_cast<char*>(workspace);
    if (p->max_len > 0) {
        st = do_score(*p, q_win, k, modality, mod_stride_b, mod_stride_h, seq_lens, lse_or_null,
                      reinterpret_cast<float*>(ws + wl.score_self), reinterpret_cast<float*>(ws + wl.score_cross),
                      workspace, stream, hist);
        if (st != CSP_OK) return st;
    }
    return launch_hist_js(*p, hist, js_or_null, js_all_or_null, stream);
}

csp_status csp_probe_ex2_rate(int32_t fma_pipe, int32_t iterations, float* sink, size_t sink_elems,
                              int64_t* exponentials_host_out, void* cuda_stream) {
    if (iterations <= 0 || iterations > (1 << 20) || !exponentials_host_out) return CSP_ERR_INVALID_ARG;
    csp_status st = check_arch();
    if (st != CSP_OK) return st;
    long long n = 0;
    st = launch_ex2_probe(fma_pipe == 2 ? 2 : (fma_pipe ? 1 : 0), iterations, sink, sink ? sink_elems : 0, &n, static_cast<cudaStream_t>(cuda_stream));
    *exponentials_host_out = n;
    return st;
}

csp_status csp_decode_attn_paged(const csp_params* p, csp_tensor q, csp_tensor k_pool, csp_tensor v_pool,
                                 const csp_pages* pages, const int32_t* n_rows, float* out, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!q.ptr || !k_pool.ptr || !v_pool.ptr || !n_rows || !out) return CSP_ERR_INVALID_ARG;
    if (p->dtype != CSP_BF16 || (p->head_dim != 64 && p->head_dim != 128)) return CSP_ERR_UNSUPPORTED;
    if (!tensor_ok(*p, q) || !tensor_ok(*p, k_pool) || !tensor_ok(*p, v_pool)) return CSP_ERR_UNSUPPORTED;
    if (!pages || !pages->page_table || pages->page_rows <= 0 || pages->page_rows % 128 || pages->max_pages <= 0 ||
        pages->n_pages <= 0 || int64_t(pages->max_pages) * pages->page_rows < p->out_capacity)
        return CSP_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < decode_workspace_bytes(*p) || (uintptr_t(workspace) % 256))
        return CSP_ERR_WORKSPACE;
    if ((st = check_arch()) != CSP_OK) return st;
    return launch_decode_attn(*p, q, k_pool, v_pool, n_rows, out, workspace, static_cast<cudaStream_t>(cuda_stream),
                              nullptr, pages);
}

size_t csp_decode_step_workspace_bytes(const csp_params* p) {
    if (check_params(p) != CSP_OK) return 0;
    return decode_step_workspace_bytes(*p);
}

csp_status csp_decode_step(const csp_params* p, csp_tensor q, csp_tensor k, csp_tensor v, const int32_t* n_rows,
                           const uint8_t* modality, int64_t mod_stride_b, int64_t mod_stride_h,
                           const uint8_t* query_label, int32_t first_step, float* out, float* acc_self,
                           float* acc_cross, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    csp_status st = check_params(p);
    if (st != CSP_OK) return st;
    if (!q.ptr || !k.ptr || !v.ptr || !n_rows || !out || !modality || !query_label || !acc_self || !acc_cross)
        return CSP_ERR_INVALID_ARG;
    if (p->dtype != CSP_BF16 || (p->head_dim != 64 && p->head_dim != 128)) return CSP_ERR_UNSUPPORTED;
    if (!tensor_ok(*p, q) || !tensor_ok(*p, k) || !tensor_ok(*p, v)) return CSP_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < decode_step_workspace_bytes(*p) || (uintptr_t(workspace) % 256))
        return CSP_ERR_WORKSPACE;
    if ((st = check_arch()) != CSP_OK) return st;
    DecodeStepArgs step = {modality, mod_stride_b, mod_stride_h, query_label, acc_self, acc_cross, first_step ? 1 : 0};
    return launch_decode_attn(*p, q, k, v, n_rows, out, workspace, static_cast<cudaStream_t>(cuda_stream), &step);
}

csp_status csp_device_status(void* workspace, void* cuda_stream, int32_t* host_out) {
    if (!workspace) return CSP_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaMemsetAsync(workspace, 0, 4, stream) != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return CSP_ERR_CUDA;
    }
    if (host_out) *host_out = word;
    return (word & CSP_DEV_TIMEOUT) ? CSP_ERR_TIMEOUT : CSP_OK;
}

const char* csp_status_string(csp_status s) {
    switch (s) {
        case CSP_OK: return "ok";
        case CSP_ERR_INVALID_ARG: return "invalid argument";
        case CSP_ERR_UNSUPPORTED: return "unsupported shape, type, stride or mode";
        case CSP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CSP_ERR_ARCH: return "device is not compute capability 10.x";
        case CSP_ERR_CUDA: return "CUDA call failed";
        case CSP_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
    }
    return "unknown status";
}

}  // extern "C"
