// pf_search.cu -- the whole search in one call: score (dense + top-k) -> survivor selection -> simulation +
// re-rank.  pf_search leaves everything on the device; pf_search_host is for callers that hold only host memory
// and adds the copies.  Inside one call the scoring kernel also collects what the selection's first pass would
// read the dense outputs for (score-bit histograms and per-chunk counts of the eligible plans), so the selection
// starts at its second pass.
#include <cstring>
#include <mutex>
#include <vector>

#include "pf_internal.cuh"

namespace pf {

// Pinned staging for the small results of pf_search_host_compact.  The caller's result pointers may be pageable
// memory, and a device-to-host copy into pageable memory blocks the host until the stream has reached it: in the
// middle of a call that would stop the host from enqueueing the rest of the search (measured: the count of feasible
// plans, copied right behind the compaction, held the selection's and the simulator's launches back by 0.2 ms).  The
// small results therefore travel into a pinned block of the library's own and are handed over with memcpy once the
// call's stream work is done.  Blocks are kept for reuse (pinning memory takes a fraction of a millisecond).
namespace {
constexpr size_t kStageBytes = 32768;
constexpr size_t kStageKeep = 8;
std::mutex g_stage_mu;
std::vector<void *> g_stage_free;
void *stage_acquire()
{
    {
        std::lock_guard<std::mutex> lock(g_stage_mu);
        if (!g_stage_free.empty()) {
            void *b = g_stage_free.back();
            g_stage_free.pop_back();
            return b;
        }
    }
    void *b = nullptr;
    if (cudaHostAlloc(&b, kStageBytes, cudaHostAllocPortable) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    return b;
}
void stage_release(void *b)
{
    if (!b) return;
    {
        std::lock_guard<std::mutex> lock(g_stage_mu);
        if (g_stage_free.size() < kStageKeep) {
            g_stage_free.push_back(b);
            return;
        }
    }
    cudaFreeHost(b);
}
// page-locked host memory (a copy into it does not block the host)?
bool host_pinned(const void *h)
{
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, h) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    return a.type == cudaMemoryTypeHost;
}
// One stream per device for pf_search_host_compact's early copy of a zero mask, shared by all plans (their copies
// share the bus anyway) and kept for the life of the process: creating and destroying a stream with every plan
// costs more than the copy saves when a plan serves a single call.
constexpr int kCopyDevices = 64;
std::mutex g_copy_mu;
cudaStream_t g_copy_stream[kCopyDevices];
cudaStream_t copy_stream_of_current_device()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kCopyDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_copy_mu);
    if (!g_copy_stream[dev] && cudaStreamCreateWithFlags(&g_copy_stream[dev], cudaStreamNonBlocking) != cudaSuccess) {
        (void)cudaGetLastError();
        g_copy_stream[dev] = nullptr;
    }
    return g_copy_stream[dev];
}
struct StageHold {   // releases the block on every return path
    void *b;
    ~StageHold() { stage_release(b); }
};
}  // namespace

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
    // sparse mode: the caller has a copy of zeros on its way to the whole host mask (done at `zeros_done`); only the
    // bits of chunks with feasible plans are written, through this device-visible alias of the host buffer
    uint8_t *mask_alias = nullptr;
    cudaEvent_t zeros_done = nullptr;
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
            if (e == cudaSuccess && cj->mask_alias) {
                e = cudaStreamWaitEvent(cs, cj->zeros_done, 0);
                if (e == cudaSuccess && compact_mask_run(p, 0, p->size, d_reason, cj->mask_alias, cj->cws, cs, guard) != PF_OK)
                    rc2 = PF_ECUDA;
            } else if (e == cudaSuccess && cj->h_mask) {
                e = cudaMemcpyAsync(cj->h_mask, cj->d_mask, ((size_t)p->size + 7) / 8, cudaMemcpyDeviceToHost, cs);
            }
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
    // the small results go through a pinned block (see stage_acquire): [histogram | count | top-k lists | simulator lists]
    StageHold hold{stage_acquire()};
    if (!hold.b) {
        set_cuda_error(cudaErrorMemoryAllocation, "pf_search_host_compact: pinned staging");
        return PF_ECUDA;
    }
    uint8_t *stage = (uint8_t *)hold.b;
    // two stretches of the device layout travel whole: the analytic top-k (indices, scores, count) and, past the
    // survivor list, the survivor count with the simulator's top-k
    const size_t tk_bytes = l.off_surv - l.off_topk_idx, sm_bytes = l.off_ws - l.off_surv_count;
    const size_t so_hist = 0, so_nfeas = PF_REASON_BINS * 8, so_tk = 256, so_sm = so_tk + tk_bytes;
    if (so_sm + sm_bytes > kStageBytes) return PF_EINVAL;   // (k, k_sim <= PF_K_MAX: 25.6 KB at most)
    uint64_t *s_hist = (uint64_t *)(stage + so_hist), *s_nfeas = (uint64_t *)(stage + so_nfeas);
    CompactJob cj;
    cj.d_hist = d_hist; cj.d_nfeas = d_nfeas; cj.d_mask = d_mask; cj.d_records = d_records; cj.record_cap = record_cap;
    cj.cws = ws + cl.off_cws;
    // the bits travel beside the search only into pinned memory; a pageable buffer gets them at the end
    const bool mask_early = h_mask && host_pinned(h_mask);
    cj.h_hist = s_hist; cj.h_nfeas = s_nfeas; cj.h_mask = mask_early ? h_mask : nullptr;
    // Nearly all of the mask is zero (a chunk of 16,384 candidates without a feasible plan: 22.5 MB for the large
    // space, of which a few hundred KB are not).  Where the device can write the host buffer directly, a copy of
    // zeros to the whole of it starts now, on a stream of its own, and crosses the bus beside the search; the
    // compact view then writes only the chunks that hold feasible plans, straight into the host buffer.
    // (Events: the plan's ev_count marks the entry for the copy stream and ev_compact the end of the zero copy; both
    // are recorded again later in the call, on the second stream, which by then has waited for this record.)
    bool zeros_forked = false;
    cudaStream_t zs = (mask_early && sim && p->side_stream) ? copy_stream_of_current_device() : nullptr;
    if (zs) {
        void *alias = nullptr;
        // (the device writes 32-bit words: a buffer that is not 4-byte aligned takes the copy at the end instead)
        if (cudaHostGetDevicePointer(&alias, h_mask, 0) == cudaSuccess && alias && ((uintptr_t)alias & 3) == 0) {
            cudaError_t e = cudaEventRecord(p->ev_count, st);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(zs, p->ev_count, 0);
            if (e == cudaSuccess) {
                zeros_forked = true;   // from here on the copy stream is joined whatever happens
                e = cudaMemsetAsync(d_mask, 0, (N + 7) / 8, zs);
                if (e == cudaSuccess) e = cudaMemcpyAsync(h_mask, d_mask, (N + 7) / 8, cudaMemcpyDeviceToHost, zs);
                const cudaError_t e2 = cudaEventRecord(p->ev_compact, zs);
                if (e == cudaSuccess) e = e2;
            }
            if (e != cudaSuccess) {
                set_cuda_error(e, "pf_search_host_compact: zero mask");
                if (zeros_forked) cudaStreamSynchronize(zs);
                return PF_ECUDA;
            }
            cj.mask_alias = (uint8_t *)alias;
            cj.zeros_done = p->ev_compact;
            cj.d_mask = nullptr;   // the compact view's kernels write no mask of their own
        } else {
            (void)cudaGetLastError();
        }
    }
    int rc = search_device(p, k, s_max, k_sim, jitter_seed, d_reason, d_tput, d_mem, d_tk_idx, d_tk_sc, d_tk_cnt,
                           d_surv, d_surv_cnt, d_sim_idx, d_sim_sc, d_sim_cnt, ws + l.off_ws, l.ws_bytes,
                           ws + l.off_ws_sel, l.ws_sel_bytes, st, &cj);
    if (zeros_forked) {
        // join the copy stream (ev_compact: the zero copy's end, or the compact view's, which waited for that)
        if (cudaStreamWaitEvent(st, p->ev_compact, 0) != cudaSuccess && rc == PF_OK) rc = PF_ECUDA;
        if (rc != PF_OK) cudaStreamSynchronize(st);   // nothing of this call touches the host buffers after it returns
    }
    if (rc != PF_OK) return rc;
    if (!cj.launched) {
        // no second stream took the compact view (a serving space, or no simulator tier): after the search
        rc = pf_compact(p, 0, N, d_reason, d_tput, d_mem, d_hist, d_mask, d_records, record_cap, d_nfeas, ws + cl.off_cws,
                        cl.cws_bytes, stream);
        if (rc != PF_OK) return rc;
        PF_CUDA_TRY(cudaMemcpyAsync(s_hist, d_hist, PF_REASON_BINS * 8, cudaMemcpyDeviceToHost, st), "copy histogram");
        PF_CUDA_TRY(cudaMemcpyAsync(s_nfeas, d_nfeas, 8, cudaMemcpyDeviceToHost, st), "copy count");
    }
    PF_CUDA_TRY(cudaMemcpyAsync(stage + so_tk, ws + l.off_topk_idx, tk_bytes, cudaMemcpyDeviceToHost, st), "copy top-k");
    if (sim) PF_CUDA_TRY(cudaMemcpyAsync(stage + so_sm, ws + l.off_surv_count, sm_bytes, cudaMemcpyDeviceToHost, st), "copy sim");
    // the record count decides how many records travel: wait for it (with a second stream at work it has been on
    // the host since shortly after the scoring kernel ended), then copy exactly those
    if (cj.launched)
        PF_CUDA_TRY(cudaEventSynchronize(p->ev_count), "pf_search_host_compact: count");
    else
        PF_CUDA_TRY(cudaStreamSynchronize(st), "pf_search_host_compact: synchronize");
    if (record_cap > 0) {
        const uint64_t n = *s_nfeas < record_cap ? *s_nfeas : record_cap;
        if (n > 0)
            PF_CUDA_TRY(cudaMemcpyAsync(h_records, d_records, (size_t)n * sizeof(pf_record_t), cudaMemcpyDeviceToHost, st),
                        "copy records");
    }
    // (a pageable h_mask or h_records makes its copy a blocking one; nothing is left to enqueue behind them)
    if (h_mask && !(cj.launched && mask_early))
        PF_CUDA_TRY(cudaMemcpyAsync(h_mask, d_mask, (N + 7) / 8, cudaMemcpyDeviceToHost, st), "copy mask");
    PF_CUDA_TRY(cudaStreamSynchronize(st), "pf_search_host_compact: synchronize");
    // hand the small results over
    memcpy(h_hist, s_hist, PF_REASON_BINS * 8);
    *h_n_feasible = *s_nfeas;
    const uint8_t *s_tk = stage + so_tk, *s_sm = stage + so_sm;
    memcpy(h_topk_idx, s_tk, (size_t)k * 8);
    memcpy(h_topk_score, s_tk + (l.off_topk_score - l.off_topk_idx), (size_t)k * 4);
    memcpy(h_topk_count, s_tk + (l.off_topk_count - l.off_topk_idx), 4);
    if (sim) {
        memcpy(h_sim_topk_idx, s_sm + (l.off_sim_idx - l.off_surv_count), (size_t)k_sim * 8);
        memcpy(h_sim_topk_score, s_sm + (l.off_sim_score - l.off_surv_count), (size_t)k_sim * 4);
        memcpy(h_sim_topk_count, s_sm + (l.off_sim_count - l.off_surv_count), 4);
        if (h_surv_count) memcpy(h_surv_count, s_sm, 8);
    } else {
        if (h_sim_topk_count) *h_sim_topk_count = 0;
        if (h_surv_count) *h_surv_count = 0;
    }
    return PF_OK;
}
