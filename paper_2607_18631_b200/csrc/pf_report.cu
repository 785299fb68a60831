// pf_report.cu -- extrapolation report for a list of plans (principle P4: a query outside the calibration domain
// of the constants is flagged, not silently trusted).  One thread re-derives one plan from its index: the reason
// byte as the scoring kernel writes it, which parts of the domain it falls outside of, its tokens per expert.
#include "pf_eval.cuh"

namespace pf {

struct ReportArgs {
    const uint64_t *idx;
    uint32_t n;
    const uint32_t *d_n;
    pf_report_t *out;
    uint64_t size;
    const int32_t *vals;
    const int32_t *scen;
};

template <typename RI>
__global__ void __launch_bounds__(128) report_kernel(const __grid_constant__ DevPlan P, const ReportArgs A)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t n = A.n;
    if (A.d_n) n = min(n, *A.d_n);
    if (i >= n) return;
    pf_report_t r;
    r.reason = 0xFF; r.why = 0; r.bucket = 0; r.reserved = 0; r.m_e = 0;
    const uint64_t idx = A.idx[i];
    if (idx < A.size) {
        int v[PF_MAX_AXES];
        uint64_t rem = idx;
#pragma unroll
        for (int a = 0; a < PF_MAX_AXES; a++) {
            const uint64_t rad = P.radix[a];
            const uint64_t q = rem / rad;
            v[a] = __ldg(A.vals + P.val_off[a] + (int)(rem - q * rad));
            rem = q;
        }
        if (P.phase == PF_PHASE_TRAIN) {
            TrainTuple c;
            c.kv = v[0]; c.rec = v[1]; c.s = v[2]; c.mb = v[3]; c.v = v[4];
            c.ep = v[5]; c.pp = v[6]; c.tp = v[7]; c.dp = v[8]; c.world = v[9];
            c.sh = P.n_axes > 10 ? v[10] : PF_SHARD_ZERO1;
            RI dp, world;
            int reason = train_layout_rules<RI>(P, c, 1, 3, dp, world);
            if (reason == 0) {
                TrainDerived<RI> D;
                D.m_e = 0;
                D.bucket = 0;
                reason = train_plan_rules<RI>(P, c, dp, world, 4, D);
                if (reason == 0 || reason >= PF_R_KERNEL_MISSING) {
                    r.m_e = (int64_t)D.m_e;
                    r.bucket = (uint16_t)D.bucket;
                }
                if (reason == 0) {
                    TrainMem M;
                    train_memory<RI>(P, c, D, M);
                    if (M.mem > P.budget_bytes) {
                        reason = PF_R_MEMORY;
                    } else {
                        r.why = (uint8_t)domain_why<RI>(P, P.kern[c.kv], D.m_e);
                        if (r.why) reason = PF_FLAG_EXTRAPOLATED;
                    }
                }
            }
            r.reason = (uint8_t)reason;
        } else {
            ServeTuple c;
            c.kv = v[0]; c.chunk = v[1]; c.batch = v[2]; c.dpa = v[3]; c.ep = v[4]; c.tp = v[5]; c.scen = v[6];
            ServeOut so;
            so.reason = 0; so.tput = 0.f; so.mem = 0;
            serve_eval<RI>(P, c, 1, __ldg(A.scen + c.scen), __ldg(A.scen + P.n_scen + c.scen), so);
            r.reason = (uint8_t)so.reason;
            r.why = (uint8_t)so.why;
            r.m_e = so.m_e;
            r.bucket = (uint16_t)so.bucket;
        }
    }
    A.out[i] = r;
}

}  // namespace pf

using namespace pf;

extern "C" int pf_report(pf_plan_t *p, const uint64_t *d_idx, uint32_t n, const uint32_t *d_n, pf_report_t *d_out,
                         void *stream)
{
    if (!p || !d_idx || !d_out) return PF_EINVAL;
    if (n == 0) return PF_OK;
    if (int rc_dev = check_device(p)) return rc_dev;
    ReportArgs a;
    a.idx = d_idx; a.n = n; a.d_n = d_n; a.out = d_out; a.size = p->size; a.vals = p->d_vals; a.scen = p->d_scen;
    const unsigned grid = (n + 127) / 128;
    cudaStream_t st = (cudaStream_t)stream;
    if (p->dev.wide)
        report_kernel<unsigned long long><<<grid, 128, 0, st>>>(p->dev, a);
    else
        report_kernel<uint32_t><<<grid, 128, 0, st>>>(p->dev, a);
    PF_CUDA_TRY(cudaGetLastError(), "report_kernel launch");
    count_launch();
    return PF_OK;
}
