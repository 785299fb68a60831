// pf_search.cu -- the whole search in one call: score (dense + top-k) -> survivor selection -> simulation +
// re-rank.  pf_search leaves everything on the device; pf_search_host is for callers that hold only host memory
// and adds the copies.  Inside one call the scoring kernel also collects what the selection's first pass would
// read the dense outputs for (score-bit histograms and per-chunk counts of the eligible plans), so the selection
// starts at its second pass.
#include "pf_internal.cuh"

namespace pf {

struct SearchLayout {
    size_t off_reason, off_tput, off_mem, off_topk_idx, off_topk_score, off_topk_count, off_surv, off_surv_count,
        off_sim_idx, off_sim_score, off_sim_count, off_ws, ws_bytes, off_ws_sel, ws_sel_bytes, total;
};

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// scratch of one search: the scoring / simulator part and the selection's part
struct WorkLayout {
    size_t ws_bytes, ws_sel_bytes, total;
};
static WorkLayout work_layout(const pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim)
{
    WorkLayout w;
    size_t a = pf_score_workspace(p, p->size, k);
    w.ws_sel_bytes = 0;
    if (s_max > 0 && p->dev.phase == PF_PHASE_TRAIN) {
        const size_t b = pf_simulate_workspace(p, s_max, k_sim);
        a = b > a ? b : a;
        w.ws_sel_bytes = align256(pf_select_workspace(p, p->size, s_max));
    }
    w.ws_bytes = align256(a);
    w.total = w.ws_bytes + w.ws_sel_bytes;
    return w;
}

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
    const WorkLayout w = work_layout(p, k, s_max, k_sim);
    l.off_ws = o;
    l.ws_bytes = w.ws_bytes;
    l.off_ws_sel = o + w.ws_bytes;
    l.ws_sel_bytes = w.ws_sel_bytes;
    l.total = o + w.total;
    return l;
}

// The compact view of a search's dense outputs (pf_compact's results) and where they go on the host: produced on the
// plan's second stream as soon as the scoring kernel is done -- every feasible plan comes from an evaluated block,
// and what the constant blocks will hold is known from their classes -- so that its copies to the host overlap with
// the selection and the simulator.
struct CompactJob {
    uint64_t *d_hist, *d_nfeas;
    uint8_t *d_mask;
    pf_record_t *d_records;
    uint64_t record_cap;
    void *cws;
    uint64_t *h_hist, *h_nfeas;
    uint8_t *h_mask;
    bool launched = false;   // out: enqueued; ev_count follows the copy of the count, ev_compact the copy of the bits
};

// The stages of one search on device buffers.  ws: scratch of the scoring call, reused by the simulator; ws_sel:
// the selection's scratch, alive from before the scoring kernel (which fills the first pass's part) to the end
// of the selection.
static int search_device(pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim, uint32_t jitter_seed,
                         uint8_t *d_reason, float *d_tput, int64_t *d_mem, uint64_t *d_tk_idx, float *d_tk_sc,
                         uint32_t *d_tk_cnt, uint64_t *d_surv, uint64_t *d_surv_cnt, uint64_t *d_sim_idx,
                         float *d_sim_sc, uint32_t *d_sim_cnt, uint8_t *ws, size_t ws_bytes, uint8_t *ws_sel,
                         size_t ws_sel_bytes, cudaStream_t st, CompactJob *cj = nullptr)
{
    const bool sim = s_max > 0 && p->dev.phase == PF_PHASE_TRAIN;
    ScoreDigest dg;
    const ScoreDigest *pdg = nullptr;
    int rc;
    if (sim) {
        rc = select_clear(p, p->size, ws_sel, ws_sel_bytes, st, &dg);
        if (rc != PF_OK) return rc;
        pdg = &dg;
    }
    // With a simulator tier to follow, the call spreads over the plan's streams.  The scoring kernel deals with the
    // evaluated slabs only (every feasible plan, the digest and the top-k keys come from those); the analytic top-k
    // is reduced on the second stream beside the selection; the constant slabs (most of the dense outputs' bytes,
    // which nothing downstream reads) are streamed by the fill kernel on the fill stream, from right behind the
    // scoring kernel to the end of the call; the fill stream joins last.  The simulator reuses the scoring scratch, so the
    // analytic top-k joins before it.
    ScoreSpread sp;
    sp.topk_aside = sim && p->side_stream != nullptr;
    sp.fill_aside = sim && p->fill_stream != nullptr;
    sp.fills_per_evaluated = sp.fill_aside ? kFillsPerEvaluatedSplit : kFillsPerEvaluated;
    rc = score_run(p, 0, p->size, d_reason, d_tput, d_mem, k, d_tk_idx, d_tk_sc, d_tk_cnt, ws, ws_bytes, st, pdg, &sp);
    bool compact_forked = false;
    if (rc == PF_OK && cj && sp.join_pending) {
        // the second stream is forked behind the scoring kernel and has the analytic top-k's reduction queued: the
        // compact view follows it there, reading evaluated blocks only while the constant ones are in flight
        cudaStream_t cs = p->side_stream;
        const FillGuard *guard = sp.fill_pending ? &sp.guard : nullptr;
        int rc2 = compact_run(p, 0, p->size, d_reason, d_tput, d_mem, cj->d_hist, cj->d_mask, cj->d_records,
                              cj->record_cap, cj->d_nfeas, cj->cws, cs, guard);
        cudaError_t e = cudaSuccess;
        if (rc2 == PF_OK) {
            e = cudaMemcpyAsync(cj->h_hist, cj->d_hist, PF_REASON_BINS * 8, cudaMemcpyDeviceToHost, cs);
            if (e == cudaSuccess) e = cudaMemcpyAsync(cj->h_nfeas, cj->d_nfeas, 8, cudaMemcpyDeviceToHost, cs);
            if (e == cudaSuccess) e = cudaEventRecord(p->ev_count, cs);
            if (e == cudaSuccess && cj->h_mask)
                e = cudaMemcpyAsync(cj->h_mask, cj->d_mask, ((size_t)p->size + 7) / 8, cudaMemcpyDeviceToHost, cs);
            if (e == cudaSuccess) e = cudaEventRecord(p->ev_compact, cs);
            if (e == cudaSuccess) cj->launched = true;
        }
        if (e != cudaSuccess) {
            set_cuda_error(e, "compact view beside the search");
            rc2 = PF_ECUDA;
        }
        // whatever was enqueued on the second stream is joined at the end of the call (below)
        if (!cj->launched && cudaEventRecord(p->ev_compact, cs) != cudaSuccess && rc2 == PF_OK) rc2 = PF_ECUDA;
        compact_forked = true;
        if (rc2 != PF_OK) rc = rc2;
    }
    if (rc == PF_OK && sim)
        rc = select_run(p, 0, p->size, d_reason, d_tput, s_max, d_surv, d_surv_cnt, ws_sel, ws_sel_bytes, st, true,
                        sp.fill_pending ? &sp.guard : nullptr);
    // joins are unconditional once a fork has happened, error returns included
    if (sp.join_pending && cudaStreamWaitEvent(st, p->ev_join, 0) != cudaSuccess && rc == PF_OK) rc = PF_ECUDA;
    if (rc == PF_OK && sim)
        rc = simulate_run(p, d_surv, s_max, d_surv_cnt, jitter_seed, nullptr, nullptr, k_sim, d_sim_idx, d_sim_sc,
                          d_sim_cnt, ws, ws_bytes, st);
    if (sp.fill_pending && cudaStreamWaitEvent(st, p->ev_fill, 0) != cudaSuccess && rc == PF_OK) rc = PF_ECUDA;
    if (compact_forked && cudaStreamWaitEvent(st, p->ev_compact, 0) != cudaSuccess && rc == PF_OK) rc = PF_ECUDA;
    return rc;
}

}  // namespace pf

using namespace pf;

extern "C" size_t pf_search_workspace(const pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim)
{
    if (!p) return 0;
    return search_layout(p, k, s_max, k_sim).total;
}

extern "C" size_t pf_search_device_workspace(const pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim)
{
    if (!p) return 0;
    return work_layout(p, k, s_max, k_sim).total;
}

extern "C" int pf_search(pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim, uint32_t jitter_seed,
                         uint8_t *d_reason, float *d_tput, int64_t *d_mem, uint64_t *d_topk_idx, float *d_topk_score,
                         uint32_t *d_topk_count, uint64_t *d_surv_idx, uint64_t *d_surv_count,
                         uint64_t *d_sim_topk_idx, float *d_sim_topk_score, uint32_t *d_sim_topk_count,
                         void *d_workspace, size_t workspace_bytes, void *stream)
{
    if (!p) return PF_EINVAL;
    if (k < 1 || k > PF_K_MAX || k_sim > PF_K_MAX) return PF_EINVAL;
    if (!d_reason || !d_tput || !d_topk_idx || !d_topk_score || !d_topk_count) return PF_EINVAL;
    if (p->size >= PF_MAX_COUNT) return PF_ERANGE;
    const bool sim = s_max > 0 && p->dev.phase == PF_PHASE_TRAIN;
    if (sim && (k_sim < 1 || !d_surv_idx || !d_surv_count || !d_sim_topk_idx || !d_sim_topk_score || !d_sim_topk_count))
        return PF_EINVAL;
    const WorkLayout w = work_layout(p, k, s_max, k_sim);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < w.total) return PF_EWORKSPACE;
    if (int rc_dev = check_device(p)) return rc_dev;
    uint8_t *ws = (uint8_t *)d_workspace;
    return search_device(p, k, s_max, k_sim, jitter_seed, d_reason, d_tput, d_mem, d_topk_idx, d_topk_score,
                         d_topk_count, d_surv_idx, d_surv_count, d_sim_topk_idx, d_sim_topk_score, d_sim_topk_count,
                         ws, w.ws_bytes, ws + w.ws_bytes, w.ws_sel_bytes, (cudaStream_t)stream);
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
    if (int rc_dev = check_device(p)) return rc_dev;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)d_workspace;
    const size_t N = (size_t)p->size;

    uint8_t *d_reason = ws + l.off_reason;
    float *d_tput = (float *)(ws + l.off_tput);
    int64_t *d_mem = h_mem ? (int64_t *)(ws + l.off_mem) : nullptr;  // not needed downstream: skip the writes
    uint64_t *d_tk_idx = (uint64_t *)(ws + l.off_topk_idx);
    float *d_tk_sc = (float *)(ws + l.off_topk_score);
    uint32_t *d_tk_cnt = (uint32_t *)(ws + l.off_topk_count);
    uint64_t *d_surv = (uint64_t *)(ws + l.off_surv);
    uint64_t *d_surv_cnt = (uint64_t *)(ws + l.off_surv_count);
    uint64_t *d_sim_idx = (uint64_t *)(ws + l.off_sim_idx);
    float *d_sim_sc = (float *)(ws + l.off_sim_score);
    uint32_t *d_sim_cnt = (uint32_t *)(ws + l.off_sim_count);
    int rc = search_device(p, k, s_max, k_sim, jitter_seed, d_reason, d_tput, d_mem, d_tk_idx, d_tk_sc, d_tk_cnt,
                           d_surv, d_surv_cnt, d_sim_idx, d_sim_sc, d_sim_cnt, ws + l.off_ws, l.ws_bytes,
                           ws + l.off_ws_sel, l.ws_sel_bytes, st);
    if (rc != PF_OK) return rc;
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

// ------------------------------------------------------------------ host buffers, compact results

namespace pf {
struct CompactSearchLayout {
    SearchLayout base;
    size_t off_hist, off_nfeas, off_mask, off_records, off_cws, cws_bytes, total;
};
static CompactSearchLayout compact_search_layout(const pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim,
                                                 uint64_t record_cap)
{
    CompactSearchLayout l;
    l.base = search_layout(p, k, s_max, k_sim);
    size_t o = l.base.total;
    l.off_hist = o; o += 256;
    l.off_nfeas = o; o += 256;
    l.off_mask = o; o += align256(((size_t)p->size + 7) / 8);
    l.off_records = o; o += align256((size_t)(record_cap ? record_cap : 1) * sizeof(pf_record_t));
    l.off_cws = o;
    l.cws_bytes = align256(pf_compact_workspace(p->size));
    l.total = o + l.cws_bytes;
    return l;
}
}  // namespace pf

extern "C" size_t pf_search_compact_workspace(const pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim,
                                              uint64_t record_cap)
{
    if (!p) return 0;
    return compact_search_layout(p, k, s_max, k_sim, record_cap).total;
}

extern "C" int pf_search_host_compact(pf_plan_t *p, uint32_t k, uint64_t s_max, uint32_t k_sim, uint32_t jitter_seed,
                                      uint64_t *h_hist, uint8_t *h_mask, pf_record_t *h_records, uint64_t record_cap,
                                      uint64_t *h_n_feasible, uint64_t *h_topk_idx, float *h_topk_score,
                                      uint32_t *h_topk_count, uint64_t *h_sim_topk_idx, float *h_sim_topk_score,
                                      uint32_t *h_sim_topk_count, uint64_t *h_surv_count, void *d_workspace,
                                      size_t workspace_bytes, void *stream)
{
    if (!p) return PF_EINVAL;
    if (k < 1 || k > PF_K_MAX || k_sim > PF_K_MAX) return PF_EINVAL;
    if (!h_hist || !h_n_feasible || !h_topk_idx || !h_topk_score || !h_topk_count) return PF_EINVAL;
    if (record_cap > 0 && !h_records) return PF_EINVAL;
    if (p->size >= PF_MAX_COUNT) return PF_ERANGE;
    const bool sim = s_max > 0 && p->dev.phase == PF_PHASE_TRAIN;
    if (sim && (k_sim < 1 || !h_sim_topk_idx || !h_sim_topk_score || !h_sim_topk_count)) return PF_EINVAL;
    const CompactSearchLayout cl = compact_search_layout(p, k, s_max, k_sim, record_cap);
    const SearchLayout &l = cl.base;
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < cl.total) return PF_EWORKSPACE;
    if (int rc_dev = check_device(p)) return rc_dev;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)d_workspace;
    const size_t N = (size_t)p->size;
    uint8_t *d_reason = ws + l.off_reason;
    float *d_tput = (float *)(ws + l.off_tput);
    int64_t *d_mem = record_cap ? (int64_t *)(ws + l.off_mem) : nullptr;   // only the records carry it
    uint64_t *d_tk_idx = (uint64_t *)(ws + l.off_topk_idx);
    float *d_tk_sc = (float *)(ws + l.off_topk_score);
    uint32_t *d_tk_cnt = (uint32_t *)(ws + l.off_topk_count);
    uint64_t *d_surv = (uint64_t *)(ws + l.off_surv);
    uint64_t *d_surv_cnt = (uint64_t *)(ws + l.off_surv_count);
    uint64_t *d_sim_idx = (uint64_t *)(ws + l.off_sim_idx);
    float *d_sim_sc = (float *)(ws + l.off_sim_score);
    uint32_t *d_sim_cnt = (uint32_t *)(ws + l.off_sim_count);
    uint64_t *d_hist = (uint64_t *)(ws + cl.off_hist), *d_nfeas = (uint64_t *)(ws + cl.off_nfeas);
    uint8_t *d_mask = h_mask ? ws + cl.off_mask : nullptr;
    pf_record_t *d_records = (pf_record_t *)(ws + cl.off_records);
    CompactJob cj;
    cj.d_hist = d_hist; cj.d_nfeas = d_nfeas; cj.d_mask = d_mask; cj.d_records = d_records; cj.record_cap = record_cap;
    cj.cws = ws + cl.off_cws;
    cj.h_hist = h_hist; cj.h_nfeas = h_n_feasible; cj.h_mask = h_mask;
    int rc = search_device(p, k, s_max, k_sim, jitter_seed, d_reason, d_tput, d_mem, d_tk_idx, d_tk_sc, d_tk_cnt,
                           d_surv, d_surv_cnt, d_sim_idx, d_sim_sc, d_sim_cnt, ws + l.off_ws, l.ws_bytes,
                           ws + l.off_ws_sel, l.ws_sel_bytes, st, &cj);
    if (rc != PF_OK) return rc;
    if (!cj.launched) {
        // no second stream took the compact view (a serving space, or no simulator tier): after the search
        rc = pf_compact(p, 0, N, d_reason, d_tput, d_mem, d_hist, d_mask, d_records, record_cap, d_nfeas, ws + cl.off_cws,
                        cl.cws_bytes, stream);
        if (rc != PF_OK) return rc;
        PF_CUDA_TRY(cudaMemcpyAsync(h_hist, d_hist, PF_REASON_BINS * 8, cudaMemcpyDeviceToHost, st), "copy histogram");
        PF_CUDA_TRY(cudaMemcpyAsync(h_n_feasible, d_nfeas, 8, cudaMemcpyDeviceToHost, st), "copy count");
        if (h_mask) PF_CUDA_TRY(cudaMemcpyAsync(h_mask, d_mask, (N + 7) / 8, cudaMemcpyDeviceToHost, st), "copy mask");
    }
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
    // the record count decides how many records travel: wait for it (with a second stream at work it has been on
    // the host since shortly after the scoring kernel ended), then copy exactly those
    if (cj.launched)
        PF_CUDA_TRY(cudaEventSynchronize(p->ev_count), "pf_search_host_compact: count");
    else
        PF_CUDA_TRY(cudaStreamSynchronize(st), "pf_search_host_compact: synchronize");
    if (record_cap > 0) {
        const uint64_t n = *h_n_feasible < record_cap ? *h_n_feasible : record_cap;
        if (n > 0)
            PF_CUDA_TRY(cudaMemcpyAsync(h_records, d_records, (size_t)n * sizeof(pf_record_t), cudaMemcpyDeviceToHost, st),
                        "copy records");
    }
    PF_CUDA_TRY(cudaStreamSynchronize(st), "pf_search_host_compact: synchronize");
    return PF_OK;
}
