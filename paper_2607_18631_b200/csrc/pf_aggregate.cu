// pf_aggregate.cu -- serving plans ranked over the whole request-length mix (Sec. 5 RQ3 compares serving
// plans): a segmented reduction of the per-(plan, scenario) scores to one score per plan, then top-k.
//
// The scenario axis is the most significant one, so the scores of plan p sit at p, p + n_plans, p + 2 n_plans,
// ...: one thread per plan walks them, and a warp's 32 plans read 32 consecutive elements of every scenario
// row (coalesced).  Traffic: 5 bytes read per candidate, 5 written per plan.
#include "pf_internal.cuh"

namespace pf {

struct AggArgs {
    const uint8_t *reason;
    const float *tput;
    uint8_t *plan_reason;
    float *plan_tput;      // never NULL inside the kernel (a workspace array stands in)
    const int32_t *scen_vals;   // scenario id per digit of the scen axis
    const int32_t *scen_O;      // output length per scenario id
    uint64_t n_plans;
    int n_digits;
};

__global__ void __launch_bounds__(256) aggregate_kernel(const AggArgs A)
{
    const uint64_t p = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= A.n_plans) return;
    int first_fail = 0, flags = 0;
    float tokens = 0.f, time = 0.f;
    for (int i = 0; i < A.n_digits; i++) {
        const uint64_t idx = p + A.n_plans * (uint64_t)i;
        const int r = A.reason[idx];
        if ((r & 0x7f) != 0) {
            if (!first_fail) first_fail = r & 0x7f;
            continue;
        }
        flags |= r & PF_FLAG_EXTRAPOLATED;
        const float O = (float)__ldg(A.scen_O + __ldg(A.scen_vals + i));
        tokens += O;
        time += __fdividef(O, A.tput[idx]);
    }
    if (A.plan_reason) A.plan_reason[p] = (uint8_t)(first_fail ? first_fail : flags);
    A.plan_tput[p] = first_fail ? 0.f : __fdividef(tokens, time);
}

struct AggLayout {
    size_t off_scores, off_topk, total;
    DenseTopkLayout dt;
};

static AggLayout agg_layout(const pf_plan_t *p, uint64_t n_plans, uint32_t k)
{
    AggLayout l;
    l.off_scores = 0;
    l.off_topk = ((size_t)(n_plans ? n_plans : 1) * 4 + 255) & ~(size_t)255;
    l.dt = dense_topk_layout(p->sm_count, n_plans, k);
    l.total = l.off_topk + (k ? l.dt.tk.total : 256);
    return l;
}

}  // namespace pf

using namespace pf;

extern "C" uint64_t pf_serve_plan_count(const pf_plan_t *p)
{
    if (!p || p->dev.phase != PF_PHASE_SERVE) return 0;
    return p->size / (uint64_t)p->dev.radix[p->dev.n_axes - 1];
}

extern "C" size_t pf_aggregate_workspace(const pf_plan_t *p, uint32_t k)
{
    if (!p || p->dev.phase != PF_PHASE_SERVE) return 0;
    return agg_layout(p, pf_serve_plan_count(p), k).total;
}

extern "C" int pf_aggregate_serving(pf_plan_t *p, const uint8_t *d_reason, const float *d_tput, uint8_t *d_plan_reason,
                                    float *d_plan_tput, uint32_t k, uint64_t *d_topk_idx, float *d_topk_score,
                                    uint32_t *d_topk_count, void *d_workspace, size_t workspace_bytes, void *stream)
{
    if (!p || !d_reason || !d_tput) return PF_EINVAL;
    if (p->dev.phase != PF_PHASE_SERVE) return PF_EUNSUPPORTED;
    if (k > PF_K_MAX) return PF_EINVAL;
    if (k > 0 && (!d_topk_idx || !d_topk_score || !d_topk_count)) return PF_EINVAL;
    const uint64_t n_plans = pf_serve_plan_count(p);
    if (n_plans >= PF_MAX_COUNT) return PF_ERANGE;
    const AggLayout lay = agg_layout(p, n_plans, k);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < lay.total) return PF_EWORKSPACE;
    if (int rc_dev = check_device(p)) return rc_dev;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)d_workspace;
    const int scen_axis = p->dev.n_axes - 1;
    AggArgs a;
    a.reason = d_reason; a.tput = d_tput; a.plan_reason = d_plan_reason;
    a.plan_tput = d_plan_tput ? d_plan_tput : (float *)(ws + lay.off_scores);
    a.scen_vals = p->d_vals + p->dev.val_off[scen_axis];
    a.scen_O = p->d_scen + p->dev.n_scen;
    a.n_plans = n_plans;
    a.n_digits = (int)p->dev.radix[scen_axis];
    timing_begin(p, PF_T_AGGREGATE, st);
    aggregate_kernel<<<(unsigned int)((n_plans + 255) / 256), 256, 0, st>>>(a);
    count_launch();
    timing_end(p, PF_T_AGGREGATE, 1, st);
    PF_CUDA_TRY(cudaGetLastError(), "aggregate_kernel launch");
    if (k > 0) {
        int nk = 0;
        timing_begin(p, PF_T_TOPK, st);
        int rc = launch_dense_topk(a.plan_tput, n_plans, nullptr, k, nullptr, ws + lay.off_topk, lay.dt, d_topk_idx,
                                   d_topk_score, d_topk_count, st, &nk);
        timing_end(p, PF_T_TOPK, nk, st);
        return rc;
    }
    return PF_OK;
}
