// pf_search.cu -- pf_search_host: the whole search for callers that hold only host memory.
// score (dense + top-k) -> survivor selection -> simulation + re-rank -> copies to the host buffers.
#include "pf_internal.cuh"

namespace pf {

struct SearchLayout {
    size_t off_reason, off_tput, off_mem, off_topk_idx, off_topk_score, off_topk_count, off_surv, off_surv_count,
        off_sim_idx, off_sim_score, off_sim_count, off_ws, ws_bytes, total;
};

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

static SearchLayout search_layout(const pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim)
{
    SearchLayout l;
    const size_t N = (size_t)p->size;
    size_t o = 0;
    l.off_reason = o; o += align256(N);
    l.off_tput = o; o += align256(N * 4);
    l.off_mem = o; o += align256(N * 8);
    l.off_topk_idx = o; o += align256((size_t)(k ? k : 1) * 8);
    l.off_topk_score = o; o += align256((size_t)(k ? k : 1) * 4);
    l.off_topk_count = o; o += 256;
    l.off_surv = o; o += align256((size_t)(s_max ? s_max : 1) * 8);
    l.off_surv_count = o; o += 256;
    l.off_sim_idx = o; o += align256((size_t)(k_sim ? k_sim : 1) * 8);
    l.off_sim_score = o; o += align256((size_t)(k_sim ? k_sim : 1) * 4);
    l.off_sim_count = o; o += 256;
    size_t w = pf_score_workspace(p, p->size, k);
    if (s_max > 0 && p->dev.phase == PF_PHASE_TRAIN) {
        size_t a = pf_select_workspace(p, p->size, s_max), b = pf_simulate_workspace(p, s_max, k_sim);
        w = a > w ? a : w;
        w = b > w ? b : w;
    }
    l.off_ws = o;
    l.ws_bytes = align256(w);
    l.total = o + l.ws_bytes;
    return l;
}

}  // namespace pf

using namespace pf;

extern "C" size_t pf_search_workspace(const pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim)
{
    if (!p) return 0;
    return search_layout(p, k, s_max, k_sim).total;
}

extern "C" int pf_search_host(pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim, uint32_t jitter_seed,
                              uint8_t *h_reason, float *h_tput, int64_t *h_mem, uint64_t *h_topk_idx,
                              float *h_topk_score, uint32_t *h_topk_count, uint64_t *h_sim_topk_idx,
                              float *h_sim_topk_score, uint32_t *h_sim_topk_count, uint64_t *h_surv_count,
                              void *d_workspace, size_t workspace_bytes, void *stream)
{
    if (!p) return PF_EINVAL;
    if (k < 1 || k > PF_K_MAX || k_sim > PF_K_MAX) return PF_EINVAL;
    if (!h_topk_idx || !h_topk_score || !h_topk_count) return PF_EINVAL;
    if (p->size >= PF_MAX_COUNT) return PF_ERANGE;
    const bool sim = s_max > 0 && p->dev.phase == PF_PHASE_TRAIN;
    if (sim && (k_sim < 1 || !h_sim_topk_idx || !h_sim_topk_score || !h_sim_topk_count)) return PF_EINVAL;
    const SearchLayout l = search_layout(p, k, s_max, k_sim);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < l.total) return PF_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)d_workspace;
    const size_t N = (size_t)p->size;

    uint8_t *d_reason = ws + l.off_reason;
    float *d_tput = (float *)(ws + l.off_tput);
    int64_t *d_mem = h_mem ? (int64_t *)(ws + l.off_mem) : nullptr;  // not needed downstream: skip the writes
    uint64_t *d_tk_idx = (uint64_t *)(ws + l.off_topk_idx);
    float *d_tk_sc = (float *)(ws + l.off_topk_score);
    uint32_t *d_tk_cnt = (uint32_t *)(ws + l.off_topk_count);
    int rc = pf_score(p, 0, p->size, d_reason, d_tput, d_mem, k, d_tk_idx, d_tk_sc, d_tk_cnt, ws + l.off_ws,
                      l.ws_bytes, stream);
    if (rc != PF_OK) return rc;
    uint64_t *d_surv = (uint64_t *)(ws + l.off_surv);
    uint64_t *d_surv_cnt = (uint64_t *)(ws + l.off_surv_count);
    uint64_t *d_sim_idx = (uint64_t *)(ws + l.off_sim_idx);
    float *d_sim_sc = (float *)(ws + l.off_sim_score);
    uint32_t *d_sim_cnt = (uint32_t *)(ws + l.off_sim_count);
    if (sim) {
        rc = pf_select_survivors(p, 0, p->size, d_reason, d_tput, s_max, d_surv, d_surv_cnt, ws + l.off_ws,
                                 l.ws_bytes, stream);
        if (rc != PF_OK) return rc;
        rc = pf_simulate(p, d_surv, s_max, d_surv_cnt, jitter_seed, nullptr, nullptr, k_sim, d_sim_idx, d_sim_sc,
                         d_sim_cnt, ws + l.off_ws, l.ws_bytes, stream);
        if (rc != PF_OK) return rc;
    }
    if (h_reason) PF_CUDA_TRY(cudaMemcpyAsync(h_reason, d_reason, N, cudaMemcpyDeviceToHost, st), "copy reason");
    if (h_tput) PF_CUDA_TRY(cudaMemcpyAsync(h_tput, d_tput, N * 4, cudaMemcpyDeviceToHost, st), "copy tput");
    if (h_mem) PF_CUDA_TRY(cudaMemcpyAsync(h_mem, d_mem, N * 8, cudaMemcpyDeviceToHost, st), "copy mem");
    PF_CUDA_TRY(cudaMemcpyAsync(h_topk_idx, d_tk_idx, (size_t)k * 8, cudaMemcpyDeviceToHost, st), "copy top-k");
    PF_CUDA_TRY(cudaMemcpyAsync(h_topk_score, d_tk_sc, (size_t)k * 4, cudaMemcpyDeviceToHost, st), "copy top-k");
    PF_CUDA_TRY(cudaMemcpyAsync(h_topk_count, d_tk_cnt, 4, cudaMemcpyDeviceToHost, st), "copy top-k");
    if (sim) {
        PF_CUDA_TRY(cudaMemcpyAsync(h_sim_topk_idx, d_sim_idx, (size_t)k_sim * 8, cudaMemcpyDeviceToHost, st), "copy sim");
        PF_CUDA_TRY(cudaMemcpyAsync(h_sim_topk_score, d_sim_sc, (size_t)k_sim * 4, cudaMemcpyDeviceToHost, st), "copy sim");
        PF_CUDA_TRY(cudaMemcpyAsync(h_sim_topk_count, d_sim_cnt, 4, cudaMemcpyDeviceToHost, st), "copy sim");
        if (h_surv_count)
            PF_CUDA_TRY(cudaMemcpyAsync(h_surv_count, d_surv_cnt, 8, cudaMemcpyDeviceToHost, st), "copy count");
    } else {
        if (h_sim_topk_count) *h_sim_topk_count = 0;
        if (h_surv_count) *h_surv_count = 0;
    }
    PF_CUDA_TRY(cudaStreamSynchronize(st), "pf_search_host: synchronize");
    return PF_OK;
}
