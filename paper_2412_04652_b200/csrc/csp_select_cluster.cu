// Selection kernel for caches up to 65536 positions: the two top-K masks (Eq. 2), their combination
// (Eq. 3) and the ascending list of kept positions followed by the recent block (index side of Eq. 4).
//
// A cluster of 1-8 CTAs owns one (sequence, KV head) unit and runs sel::select_unit on it (radix select
// with the keys in registers; see csp_select_unit.cuh).  Many warps with little code each hide the
// latencies of the short dependent phases better than few fat threads.
#include "csp_select_unit.cuh"

namespace csp {
namespace {

template <int kCsThreads, int E>
__global__ void __launch_bounds__(kCsThreads, kCsThreads <= 256 ? 4 : (kCsThreads <= 512 ? 2 : 1))
select_cluster_kernel(const SelectArgs a) {
    __shared__ sel::SelectSmem<kCsThreads / 32> sm;
    sel::select_unit<kCsThreads, E, false>(a, blockIdx.y, sm);
}

template <int kCsThreads, int E>
csp_status launch_e(const csp_params& p, const SelectArgs& a, int cs, cudaStream_t s) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cs, p.batch * p.n_kv_heads, 1);
    cfg.blockDim = dim3(kCsThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, select_cluster_kernel<kCsThreads, E>, a) != cudaSuccess) { cudaGetLastError(); return CSP_ERR_CUDA; }
    return CSP_OK;
}

}  // namespace

csp_status launch_select_cluster(const csp_params& p, const SelectArgs& a, cudaStream_t s) {
    const int units = p.batch * p.n_kv_heads;
    if (units == 0) return CSP_OK;
    if (units > 65535) return CSP_ERR_UNSUPPORTED;
    // A CTA covers 4096 keys, or 8192 for caches above 4096 positions: smaller clusters mean fewer cluster
    // barriers per round and, in a ragged batch, fewer CTAs that hold no keys.  With many units the CTAs have
    // 512 threads (8 or 16 keys per thread), two per SM, so that one CTA's barrier phases overlap the other's work.
    // Short caches (the re-prune rounds of a serving batch: a few hundred rows per head) take small CTAs, so that
    // a whole batch of units is resident at once instead of queueing in waves of two CTAs per SM.
    if (p.max_len <= 512) return launch_e<256, 2>(p, a, 1, s);
    if (p.max_len <= 1024) return launch_e<256, 4>(p, a, 1, s);
    if (p.max_len <= 2048) return launch_e<512, 4>(p, a, 1, s);
    const int per_cta = p.max_len <= 4096 ? 4096 : 8192;
    int cs = 1;
    while (cs < 8 && cs * per_cta < p.max_len) cs *= 2;
    const int sms = sm_count();
    if (per_cta == 8192) return units * cs >= 2 * sms ? launch_e<512, 16>(p, a, cs, s) : launch_e<1024, 8>(p, a, cs, s);
    if (units * cs >= 2 * sms) return launch_e<512, 8>(p, a, cs, s);
    return launch_e<1024, 4>(p, a, cs, s);
}

}  // namespace csp
