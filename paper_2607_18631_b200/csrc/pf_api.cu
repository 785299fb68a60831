// pf_api.cu -- handle life cycle, validation, host-side derivation of the candidate-independent constants,
// status strings.  Host code only.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "pf_internal.cuh"

namespace pf {

static thread_local char g_cuda_msg[256] = "";
static std::atomic<uint64_t> g_launches{0};

void set_cuda_error(cudaError_t e, const char *where)
{
    snprintf(g_cuda_msg, sizeof(g_cuda_msg), "%s: %s", where, cudaGetErrorString(e));
}
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

int check_device(const pf_plan_t *p)
{
    int dev = -1;
    PF_CUDA_TRY(cudaGetDevice(&dev), "current device");
    if (dev != p->device) {
        snprintf(g_cuda_msg, sizeof(g_cuda_msg), "the plan belongs to device %d, the current device is %d", p->device, dev);
        return PF_EINVAL;
    }
    return PF_OK;
}

struct TimingRec {
    int cls, n_kernels;
    bool open;
    cudaEvent_t a, b;
};
struct Timing {
    bool on = false;
    uint32_t mask = ~0u;   // classes that are timed
    uint32_t every = 1;    // ... in every `every`-th of their launch groups
    uint32_t seen[PF_T_CLASSES] = {};
    std::vector<TimingRec> recs;
    std::vector<cudaEvent_t> pool;
    cudaEvent_t get()
    {
        if (!pool.empty()) {
            cudaEvent_t e = pool.back();
            pool.pop_back();
            return e;
        }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
};

void timing_begin(pf_plan_t *p, int cls, cudaStream_t st)
{
    Timing *t = (Timing *)p->timing;
    if (!t || !t->on || !((t->mask >> cls) & 1u)) return;
    if (t->seen[cls]++ % t->every != 0) return;   // (timing_end finds no open record of the class and does nothing)
    TimingRec r;
    r.cls = cls;
    r.n_kernels = 0;
    r.open = true;
    r.a = t->get();
    r.b = t->get();
    cudaEventRecord(r.a, st);
    t->recs.push_back(r);
}

void timing_end(pf_plan_t *p, int cls, int n_kernels, cudaStream_t st)
{
    Timing *t = (Timing *)p->timing;
    if (!t || !t->on || !((t->mask >> cls) & 1u)) return;
    // the latest open record of this class (records of classes launched on other streams may lie in between)
    for (size_t i = t->recs.size(); i-- > 0;) {
        TimingRec &r = t->recs[i];
        if (r.cls != cls || !r.open) continue;
        r.open = false;
        r.n_kernels = n_kernels;
        cudaEventRecord(r.b, st);
        return;
    }
}

}  // namespace pf

using pf::DevPlan;

namespace pf {
// ------------------------------------------------------------------ dynamic shared-memory limits
namespace {
constexpr int kSmemDevices = 64;
struct SmemLimit {
    const void *kernel;
    size_t have[kSmemDevices];
};
std::mutex g_smem_mu;
std::vector<SmemLimit> g_smem;   // a handful of kernels: a linear search
}  // namespace

cudaError_t ensure_dynamic_smem(const void *kernel, int device, size_t bytes)
{
    if (device < 0 || device >= kSmemDevices) return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    std::lock_guard<std::mutex> lock(g_smem_mu);
    SmemLimit *l = nullptr;
    for (SmemLimit &x : g_smem)
        if (x.kernel == kernel) l = &x;
    if (!l) {
        g_smem.push_back(SmemLimit{kernel, {}});
        l = &g_smem.back();
    }
    if (l->have[device] >= bytes) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) l->have[device] = bytes;
    return e;
}

// ------------------------------------------------------------------ per-device caches of plan resources
// A plan owns one block of device memory, two streams and six events.  Creating and releasing those through the
// runtime takes 0.3 - 0.9 ms per plan (measured), several times the search of a large space, so released ones are
// kept -- a few per device, blocks only up to kArenaKeepBytes -- and handed to the next plan.  A block is handed back
// only after the device has gone idle (pf_plan_destroy), so nothing of its former plan can still touch it.
namespace {
constexpr size_t kArenaKeepBytes = 8u << 20;
constexpr size_t kKeepPerDevice = 4;
struct ArenaSlot {
    int device;
    void *base;
    size_t cap;
};
struct StreamSlot {
    int device;
    cudaStream_t side, fill;
    cudaEvent_t ev[6];
};
std::mutex g_cache_mu;
std::vector<ArenaSlot> g_arenas;
std::vector<StreamSlot> g_streams;
}  // namespace

void *arena_acquire(int device, size_t need, size_t *cap)
{
    {
        std::lock_guard<std::mutex> lock(g_cache_mu);
        for (size_t i = 0; i < g_arenas.size(); i++)
            if (g_arenas[i].device == device && g_arenas[i].cap >= need) {
                void *b = g_arenas[i].base;
                *cap = g_arenas[i].cap;
                g_arenas.erase(g_arenas.begin() + (long)i);
                return b;
            }
    }
    void *b = nullptr;
    // (rounded up so that plans of similar spaces can take each other's blocks)
    const size_t want = (need + 65535) & ~(size_t)65535;
    if (cudaMalloc(&b, want) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    *cap = want;
    return b;
}

void arena_release(int device, void *base, size_t cap)
{
    if (!base) return;
    if (cap <= kArenaKeepBytes) {
        std::lock_guard<std::mutex> lock(g_cache_mu);
        size_t kept = 0;
        for (const ArenaSlot &a : g_arenas) kept += a.device == device;
        if (kept < kKeepPerDevice) {
            g_arenas.push_back(ArenaSlot{device, base, cap});
            return;
        }
    }
    cudaFree(base);
}

cudaError_t streams_acquire(pf_plan_t *p)
{
    {
        std::lock_guard<std::mutex> lock(g_cache_mu);
        for (size_t i = 0; i < g_streams.size(); i++)
            if (g_streams[i].device == p->device) {
                const StreamSlot s = g_streams[i];
                g_streams.erase(g_streams.begin() + (long)i);
                p->side_stream = s.side; p->fill_stream = s.fill;
                p->ev_fork = s.ev[0]; p->ev_join = s.ev[1]; p->ev_fill = s.ev[2];
                p->ev_fork3 = s.ev[3]; p->ev_count = s.ev[4]; p->ev_compact = s.ev[5];
                return cudaSuccess;
            }
    }
    // the fill stream carries a long streaming kernel that should yield to everything else: lowest priority
    int prio_lo = 0, prio_hi = 0;
    cudaError_t e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&p->side_stream, cudaStreamNonBlocking, prio_hi);
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&p->fill_stream, cudaStreamNonBlocking, prio_lo);
    cudaEvent_t *evs[6] = {&p->ev_fork, &p->ev_join, &p->ev_fill, &p->ev_fork3, &p->ev_count, &p->ev_compact};
    for (int i = 0; i < 6 && e == cudaSuccess; i++) e = cudaEventCreateWithFlags(evs[i], cudaEventDisableTiming);
    return e;   // on failure pf_plan_destroy releases what was created
}

void streams_release(pf_plan_t *p)
{
    const bool complete = p->side_stream && p->fill_stream && p->ev_fork && p->ev_join && p->ev_fill && p->ev_fork3 &&
                          p->ev_count && p->ev_compact;
    if (complete) {
        std::lock_guard<std::mutex> lock(g_cache_mu);
        size_t kept = 0;
        for (const StreamSlot &s : g_streams) kept += s.device == p->device;
        if (kept < kKeepPerDevice) {
            g_streams.push_back(StreamSlot{p->device, p->side_stream, p->fill_stream,
                                           {p->ev_fork, p->ev_join, p->ev_fill, p->ev_fork3, p->ev_count, p->ev_compact}});
            p->side_stream = p->fill_stream = nullptr;
            p->ev_fork = p->ev_join = p->ev_fill = p->ev_fork3 = p->ev_count = p->ev_compact = nullptr;
            return;
        }
    }
    cudaEvent_t evs[6] = {p->ev_fork, p->ev_join, p->ev_fill, p->ev_fork3, p->ev_count, p->ev_compact};
    for (cudaEvent_t ev : evs)
        if (ev) cudaEventDestroy(ev);
    if (p->side_stream) cudaStreamDestroy(p->side_stream);
    if (p->fill_stream) cudaStreamDestroy(p->fill_stream);
    p->side_stream = p->fill_stream = nullptr;
    p->ev_fork = p->ev_join = p->ev_fill = p->ev_fork3 = p->ev_count = p->ev_compact = nullptr;
}

int build_sim_tables(pf_plan_t *p);  // pf_simulate.cu: schedule-order tables for the simulator (host part)
size_t sim_tables_bytes(const pf_plan_t *p);
void sim_tables_place(pf_plan_t *p, uint8_t *dev, uint8_t *image);
void free_sim_tables(pf_plan_t *p);
}

extern "C" int pf_version(void) { return PF_VERSION; }

extern "C" const char *pf_last_cuda_error(void) { return pf::g_cuda_msg; }

extern "C" uint64_t pf_launch_count(void) { return pf::g_launches.load(); }

extern "C" const char *pf_strerror(int status)
{
    switch (status) {
    case PF_OK: return "ok";
    case PF_EINVAL: return "invalid argument";
    case PF_ERANGE: return "value out of range";
    case PF_EWORKSPACE: return "workspace too small or misaligned";
    case PF_ECUDA: return "CUDA error";
    case PF_EUNSUPPORTED: return "not supported for this plan";
    default: return "unknown status";
    }
}

extern "C" const char *pf_reason_str(uint8_t reason)
{
    switch (reason & 0x7f) {
    case PF_FEASIBLE: return (reason & PF_FLAG_EXTRAPOLATED) ? "feasible (extrapolated)" : "feasible";
    case PF_R_WORLD: return "world size does not match the parallel degrees";
    case PF_R_TP: return "tensor-parallel degree not admissible";
    case PF_R_EP: return "expert-parallel degree not admissible";
    case PF_R_BATCH: return "global batch not divisible by dp * microbatch";
    case PF_R_VSTAGE: return "virtual-stage count does not fit the schedule class";
    case PF_R_LAYERS: return "layer count does not divide the pipeline depth";
    case PF_R_MICROBATCH: return "microbatch count does not fit the schedule order";
    case PF_R_KERNEL_MISSING: return "kernel variant missing for this expert shape or hardware";
    case PF_R_UNMAPPED_SCHEDULE: return "schedule class has no realization in the toolchain";
    case PF_R_OVERLAP_PRECOND: return "overlap precondition violated";
    case PF_R_MEMORY: return "memory_infeasible";
    default: return "unknown reason";
    }
}

// Per-layer parameter, activation and FLOP counts (exact int64 on the host).
static void derive_model(const pf_model_t &m, DevPlan &d)
{
    const long long H = m.H, nh = m.nh, nkv = m.nkv, hd = m.hd, ab = m.ab;
    const long long lat = m.kv_latent, rope = m.rope_dim;
    const bool mla = m.attn_kind != 0;
    d.dk = mla ? (int)(lat + rope) : m.hd;
    const long long hq = m.hd_q > 0 ? m.hd_q : hd;
    const long long q_proj = H * nh * hq, o_proj = nh * hd * H;
    if (!mla)
        d.P_attn = q_proj + 2 * H * nkv * hd + o_proj;
    else
        d.P_attn = q_proj + H * (lat + rope) + lat * nh * 2 * hd + o_proj;
    d.P_rt = H * (long long)m.E;
    d.P_e = (long long)m.n_mats * H * m.F;
    d.P_sh = (long long)m.S * m.n_mats * H * m.Fs;
    d.P_dl = d.P_attn + d.P_sh;
    d.P_emb = m.count_embeddings ? (long long)m.vocab * H : 0;

    const long long qkv = mla ? nh * hd + lat + rope + 2 * nh * hd : (nh + 2 * nkv) * hd;
    const long long a_attn = ab * (2 * H + qkv + nh * hd);
    const long long a_fix = ab * 2 * H + 4ll * m.E + ab * m.K * H + ab * H;
    const long long a_ffn = ab * 3 * ((long long)m.K * m.F + (long long)m.S * m.Fs);
    d.a_full = a_attn + a_fix + a_ffn;
    d.a_sel = a_attn + a_fix;
    d.a_ckpt = ab * H;

    const long long f_attn = 2 * d.P_attn + 2ll * m.seq * nh * d.dk;
    const long long f_rt = 2 * H * (long long)m.E;
    const long long f_sh = 2 * d.P_sh;
    d.f_dense = (float)(f_attn + f_rt + f_sh);
    d.f_exp = (float)(2ll * m.K * d.P_e);
    d.f_head = (float)(2ll * m.vocab * H);
    d.f_sh = (float)f_sh;

    // a leading dense layer: attention + a plain FFN, no router, no experts
    d.L_dense = m.L_dense;
    d.P_dld = d.P_attn + (long long)m.n_mats * H * m.F_dense;
    d.a_sel_d = a_attn + ab * 2 * H;
    d.a_full_d = d.a_sel_d + ab * 3 * (long long)m.F_dense;
    const long long f_mlp_d = 2ll * m.n_mats * H * m.F_dense;
    d.f_mlp_d = (float)f_mlp_d;
    d.f_dense_d = (float)(f_attn + f_mlp_d);
}

static bool positive(std::initializer_list<long long> xs)
{
    for (long long x : xs)
        if (x <= 0) return false;
    return true;
}

extern "C" int pf_plan_create(const pf_model_t *model, const pf_cluster_t *cluster, const pf_workload_t *workload,
                              const pf_axes_t *axes, const pf_tables_t *tables, const pf_rules_t *rules,
                              pf_plan_t **out)
{
    if (!model || !cluster || !workload || !axes || !tables || !rules || !out) return PF_EINVAL;
    *out = nullptr;
    const int phase = workload->phase;
    if (phase != PF_PHASE_TRAIN && phase != PF_PHASE_SERVE) return PF_EINVAL;
    // training spaces may carry the memory-sharding axis as an 11th, most significant one
    const int want_axes = phase == PF_PHASE_TRAIN ? (axes->n_axes == 11 ? 11 : 10) : 7;
    if (axes->n_axes != want_axes) return PF_EINVAL;
    if (tables->n_sched < 1 || tables->n_sched > PF_MAX_SCHED || tables->n_kern < 1 || tables->n_kern > PF_MAX_KERN)
        return PF_EINVAL;
    const pf_model_t &M = *model;
    if (!positive({M.L, M.H, M.nh, M.hd, M.E, M.K, M.F, M.seq, M.vocab, M.wb, M.gb, M.ob, M.ab, M.n_mats}))
        return PF_EINVAL;
    if (M.S < 0 || (M.S > 0 && M.Fs <= 0) || M.K > M.E) return PF_EINVAL;
    if (M.L_dense < 0 || M.L_dense >= M.L || (M.L_dense > 0 && M.F_dense <= 0) || M.F_dense < 0 || M.hd_q < 0)
        return PF_EINVAL;
    if (M.attn_kind == 0 ? M.nkv <= 0 : (M.kv_latent <= 0 || M.rope_dim < 0)) return PF_EINVAL;
    if (cluster->G <= 0 || cluster->budget_bytes < 0 || cluster->reserved_bytes < 0) return PF_EINVAL;
    if (!(cluster->peak_flops > 0) || !(cluster->hbm_bw > 0) || !(cluster->bw_intra > 0) || !(cluster->bw_inter > 0))
        return PF_EINVAL;
    if (want_axes == 11 && (!(cluster->bw_host > 0) || !(tables->offload_overlap_penalty > -1.f))) return PF_EINVAL;
    if (!(tables->eff_dense > 0) || !(tables->dualpipe_startup_div > 0)) return PF_EINVAL;
    if (phase == PF_PHASE_TRAIN && workload->gbs <= 0) return PF_EINVAL;
    if (phase == PF_PHASE_SERVE) {
        if (workload->world <= 0 || workload->n_scen < 1 || workload->n_scen > PF_MAX_SCEN) return PF_EINVAL;
        if (!workload->scen_P || !workload->scen_O) return PF_EINVAL;
        for (int i = 0; i < workload->n_scen; i++)
            if (workload->scen_P[i] < 1 || workload->scen_O[i] < 1) return PF_ERANGE;
    }

    // axes: lengths, packed values, space size
    int total_vals = 0;
    uint64_t N = 1;
    for (int a = 0; a < want_axes; a++) {
        int len = axes->len[a];
        if (len < 1 || len > PF_MAX_AXIS_LEN) return PF_ERANGE;
        if (!axes->val[a]) return PF_EINVAL;
        if (N > (UINT64_MAX >> 1) / (uint64_t)len) return PF_ERANGE;  // keep N < 2^63
        N *= (uint64_t)len;
        total_vals += len;
    }
    // value ranges per axis
    auto in_range = [&](int a, long long lo, long long hi) {
        for (int i = 0; i < axes->len[a]; i++)
            if (axes->val[a][i] < lo || axes->val[a][i] > hi) return false;
        return true;
    };
    const long long kDeg = 1 << 20;  // largest parallel degree / world size the integer paths are sized for
    bool dp_derived = false, world_derived = false;
    if (phase == PF_PHASE_TRAIN) {
        if (!in_range(0, 0, tables->n_kern - 1) || !in_range(1, 0, 2) || !in_range(2, 0, tables->n_sched - 1))
            return PF_EINVAL;
        if (!in_range(3, 1, 1 << 16) || !in_range(4, 0, 255)) return PF_ERANGE;
        if (!in_range(5, 1, kDeg) || !in_range(6, 1, kDeg) || !in_range(7, 1, kDeg)) return PF_ERANGE;
        if (!in_range(8, 0, kDeg) || !in_range(9, 0, kDeg)) return PF_ERANGE;
        if (want_axes == 11 && !in_range(10, PF_SHARD_ZERO1, PF_SHARD_FSDP)) return PF_EINVAL;
        // "derived" is a whole-axis statement: the list {0}
        for (int a = 8; a <= 9; a++) {
            bool has0 = false;
            for (int i = 0; i < axes->len[a]; i++) has0 |= axes->val[a][i] == 0;
            if (has0 && axes->len[a] != 1) return PF_EINVAL;
            (a == 8 ? dp_derived : world_derived) = has0;
        }
        if (dp_derived && world_derived) return PF_EINVAL;
        {
            bool has0 = false;
            for (int i = 0; i < axes->len[4]; i++) has0 |= axes->val[4][i] == 0;
            if (has0 && axes->len[4] != 1) return PF_EINVAL;
        }
        for (int s = 0; s < tables->n_sched; s++)
            if (tables->sched[s].kind < 0 || tables->sched[s].kind > 2 || tables->sched[s].n_chunks < 0 ||
                tables->sched[s].n_chunks > 16 || !(tables->sched[s].sm_frac >= 0.f) || tables->sched[s].sm_frac > 0.9f)
                return PF_EINVAL;
    } else {
        if (!in_range(0, 0, tables->n_kern - 1)) return PF_EINVAL;
        if (!in_range(1, 1, 1 << 20) || !in_range(2, 1, 1 << 20) || !in_range(3, 0, 1)) return PF_ERANGE;
        if (!in_range(4, 1, kDeg) || !in_range(5, 1, kDeg)) return PF_ERANGE;
        if (!in_range(6, 0, workload->n_scen - 1)) return PF_EINVAL;
    }
    for (int i = 0; i < tables->n_kern; i++) {
        const pf_kern_t &k = tables->kern[i];
        if (!(k.dtype_mult > 0) || k.wbytes < 1 || k.dtype < 0 || k.dtype > 31) return PF_EINVAL;
        for (int b = 0; b < PF_NBUCKET; b++)
            if (!(k.eff[b] > 0)) return PF_EINVAL;
    }

    pf_plan_t *p = new (std::nothrow) pf_plan_t;
    if (!p) return PF_EINVAL;
    memset(p, 0, sizeof(*p));
    DevPlan &d = p->dev;
    p->size = N;
    d.phase = phase;
    d.n_axes = want_axes;

    // packed values
    p->h_vals = (int32_t *)malloc(sizeof(int32_t) * (size_t)total_vals);
    int off = 0;
    for (int a = 0; a < want_axes; a++) {
        p->axis_len[a] = axes->len[a];
        d.radix[a] = (uint32_t)axes->len[a];
        d.val_off[a] = off;
        memcpy(p->h_vals + off, axes->val[a], sizeof(int32_t) * (size_t)axes->len[a]);
        off += axes->len[a];
    }
    // axes the space does not have decode as a single digit 0 that reads the first packed value
    for (int a = want_axes; a < PF_MAX_AXES; a++) {
        p->axis_len[a] = 1;
        d.radix[a] = 1;
        d.val_off[a] = 0;
    }

    // slab = longest axis prefix whose product stays under a size that still leaves a few blocks per SM
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {   // (the full property
        pf::set_cuda_error(cudaGetLastError(), "pf_plan_create: device query");           // query takes a millisecond)
        free(p->h_vals);
        delete p;
        return PF_ECUDA;
    }
    p->device = dev;
    p->sm_count = sms;
    uint64_t target = N / (uint64_t)(4 * p->sm_count);
    if (target < 256) target = 256;
    if (target > pf::kSlabMax) target = pf::kSlabMax;
    uint64_t slab = 1;
    int n_inner = 0;
    while (n_inner < want_axes && slab * d.radix[n_inner] <= target) {
        slab *= d.radix[n_inner];
        n_inner++;
    }
    // a first axis longer than the target still makes a better slab than single candidates
    if (n_inner == 0 && d.radix[0] <= pf::kSlabMax) {
        slab = d.radix[0];
        n_inner = 1;
    }
    d.n_inner = n_inner;
    d.slab = (uint32_t)slab;
    for (int a = 0; a < want_axes; a++) {
        // ceil(2^32 / r): exact quotient by multiply-high for n < 2^32 / r, and n <= slab * ... <= 2^14
        d.magic[a] = d.radix[a] == 1 ? 0u : (uint32_t)(((1ull << 32) + d.radix[a] - 1) / d.radix[a]);
    }
    // Per-slab table of rules 4-7 (batch, virtual stages, layers, microbatches): they depend on the layout
    // and on (sched, mb, v) only, so when the layout axes are all outer a slab evaluates them once per
    // (sched, mb, v) combination instead of once per candidate.
    d.tab_n[0] = d.tab_n[1] = d.tab_n[2] = 0;
    if (phase == PF_PHASE_TRAIN && n_inner <= 5) {
        uint64_t n2 = n_inner > 2 ? d.radix[2] : 1, n3 = n_inner > 3 ? d.radix[3] : 1, n4 = n_inner > 4 ? d.radix[4] : 1;
        if (n2 * n3 * n4 <= 2048) d.tab_n[0] = (int)n2, d.tab_n[1] = (int)n3, d.tab_n[2] = (int)n4;
    }
    // leading rules whose axes are all outer (train: R1 tp,pp,dp,world; R2 tp; R3 ep,dp,tp; R4 dp,mb;
    // serve: R1 tp,dpa,ep; R2 tp; R3 ep,tp,dpa; R4 dpa,batch,ep)
    if (phase == PF_PHASE_TRAIN)
        d.n_pre_rules = n_inner <= 3 ? 4 : n_inner <= 5 ? 3 : n_inner <= 6 ? 2 : 0;
    else
        d.n_pre_rules = n_inner <= 2 ? 4 : n_inner <= 3 ? 3 : 0;

    // model, cluster, workload, tables
    d.L = M.L; d.H = M.H; d.nh = M.nh; d.nkv = M.nkv; d.hd = M.hd; d.attn_kind = M.attn_kind;
    d.kv_latent = M.kv_latent; d.rope_dim = M.rope_dim; d.E = M.E; d.K = M.K; d.F = M.F; d.S = M.S; d.Fs = M.Fs;
    d.seq = M.seq; d.vocab = M.vocab; d.wb = M.wb; d.gb = M.gb; d.ob = M.ob; d.ab = M.ab;
    d.count_embeddings = M.count_embeddings ? 1 : 0;
    derive_model(M, d);
    d.G = cluster->G; d.caps = cluster->caps;
    d.budget_bytes = cluster->budget_bytes; d.reserved_bytes = cluster->reserved_bytes;
    d.peak_flops = cluster->peak_flops; d.hbm_bw = cluster->hbm_bw;
    d.bw_intra = cluster->bw_intra; d.bw_inter = cluster->bw_inter;
    d.alpha_intra = cluster->alpha_intra; d.alpha_inter = cluster->alpha_inter;
    d.bw_host = cluster->bw_host; d.offload_overlap_penalty = tables->offload_overlap_penalty;
    d.gpu_id = cluster->gpu_id;
    d.dom_attached = tables->domain.attached ? 1 : 0; d.dom_gpu = tables->domain.gpu_id;
    d.dom_dtypes = tables->domain.dtype_mask; d.dom_m_lo = tables->domain.m_lo; d.dom_m_hi = tables->domain.m_hi;
    d.gbs = workload->gbs; d.world = workload->world; d.n_scen = phase == PF_PHASE_SERVE ? workload->n_scen : 0;
    d.eff_dense = tables->eff_dense; d.bwd_factor = tables->bwd_factor; d.dp_overlap_frac = tables->dp_overlap_frac;
    d.dualpipe_startup_div = tables->dualpipe_startup_div; d.step_overhead = tables->step_overhead;
    d.ep_scope = rules->ep_scope ? 1 : 0; d.layer_mode = rules->layer_mode; d.tp_max = rules->tp_max;
    d.world_min = rules->world_min; d.world_max = rules->world_max;
    d.enforce = rules->enforce_realizability ? 1 : 0;
    d.n_sched = tables->n_sched; d.n_kern = tables->n_kern;
    for (int s = 0; s < tables->n_sched; s++) {
        d.sched[s].kind = tables->sched[s].kind; d.sched[s].overlap = tables->sched[s].overlap ? 1 : 0;
        d.sched[s].mapped = tables->sched[s].mapped ? 1 : 0;
        d.sched[s].hide_frac = tables->sched[s].hide_frac; d.sched[s].sched_ovh = tables->sched[s].sched_ovh;
        d.sched[s].n_chunks = tables->sched[s].n_chunks; d.sched[s].sm_frac = tables->sched[s].sm_frac;
    }
    for (int i = 0; i < tables->n_kern; i++) {
        const pf_kern_t &k = tables->kern[i];
        d.kern[i].needs_caps = k.needs_caps; d.kern[i].avail_mask = k.avail_mask;
        d.kern[i].is_native = k.is_native ? 1 : 0; d.kern[i].wbytes = k.wbytes;
        d.kern[i].dtype_mult = k.dtype_mult; d.kern[i].patch_ovh = k.patch_ovh;
        for (int b = 0; b < PF_NBUCKET; b++) d.kern[i].eff[b] = k.eff[b];
        d.kern[i].dtype = k.dtype;
    }

    // can the rule arithmetic stay in 32 bits?  (largest products the rules form)
    auto axis_max = [&](int a) {
        long long m = 0;
        for (int i = 0; i < axes->len[a]; i++) m = axes->val[a][i] > m ? axes->val[a][i] : m;
        return m;
    };
    const long long lim = (1ll << 31) - 1;
    bool wide = false;
    if (phase == PF_PHASE_TRAIN) {
        long long mb = axis_max(3), ep = axis_max(5), pp = axis_max(6), tp = axis_max(7);
        long long dp = dp_derived ? axis_max(9) : axis_max(8);
        long long world = world_derived ? tp * pp * dp : axis_max(9);
        wide |= tp * pp > lim || tp * pp * dp > lim || world > lim || dp * tp > lim || dp * mb > lim;
        wide |= workload->gbs > lim || mb * M.seq > lim || mb * M.seq * M.K > lim / (ep > 0 ? ep : 1);
        wide |= (long long)M.E * tp > lim || pp * 256 > lim;
    } else {
        long long C = axis_max(1), B = axis_max(2), ep = axis_max(4), tp = axis_max(5);
        wide |= tp * ep > lim || B * M.K > lim || C * M.K > lim || workload->world > lim;
    }
    d.wide = wide ? 1 : 0;
    // A feasible training plan has pp * v <= L (layer rule).  If no listed pp or v value that can pass that
    // rule leaves the simulator's domain, survivor selection needs no per-candidate domain check.
    d.sim_domain_all = 0;
    if (phase == PF_PHASE_TRAIN) {
        bool all_in = true;
        for (int i = 0; i < axes->len[6]; i++) {
            int pp = axes->val[6][i];
            if (pp <= M.L && pp > PF_SIM_MAX_RANKS) all_in = false;
        }
        for (int i = 0; i < axes->len[4]; i++) {
            int v = axes->val[4][i] == 0 ? 2 : axes->val[4][i];
            if (v <= M.L && v > PF_SIM_MAX_V) all_in = false;
        }
        d.sim_domain_all = all_in ? 1 : 0;
    }

    // Device side: ONE block per plan -- [axis values | scenario lengths | fill-kernel control | check record |
    // simulator order tables | order-table header] uploaded as one image, then the order table's body, which the
    // first call builds.  The block comes from a small per-device cache (see arena_acquire), and so do the plan's
    // streams and events: a plan that serves a single call would otherwise spend more time in the allocator
    // than in the search.
    if (phase == PF_PHASE_TRAIN) {
        int rc = pf::build_sim_tables(p);
        if (rc != PF_OK) {
            pf_plan_destroy(p);
            return rc;
        }
    }
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t n_scen = phase == PF_PHASE_SERVE ? (size_t)workload->n_scen : 0;
    const size_t o_vals = 0, o_scen = o_vals + up(sizeof(int32_t) * (size_t)total_vals);
    const size_t o_fill = o_scen + up(sizeof(int32_t) * 2 * n_scen), o_check = o_fill + 2048, o_sim = o_check + 256;
    const size_t o_order = o_sim + pf::sim_tables_bytes(p);
    // room for the slab visiting order of one pf_score range (any alignment of its first candidate)
    const uint64_t slabs = (p->size + d.slab - 1) / d.slab + 1;
    const bool has_order = slabs <= (uint64_t)pf::kOrderMaxSlabs;
    const size_t image_bytes = o_order + 256;
    const size_t need = has_order ? o_order + up(256 + (size_t)slabs * 5) : image_bytes;
    p->arena = pf::arena_acquire(dev, need, &p->arena_cap);
    if (!p->arena) {
        pf::set_cuda_error(cudaErrorMemoryAllocation, "pf_plan_create: device block");
        pf_plan_destroy(p);
        return PF_ECUDA;
    }
    uint8_t *base = (uint8_t *)p->arena;
    p->d_vals = (int32_t *)(base + o_vals);
    if (n_scen) p->d_scen = (int32_t *)(base + o_scen);
    p->d_fill_ctl = (unsigned int *)(base + o_fill);
    p->d_check = (unsigned int *)(base + o_check);
    d.chk = p->d_check;
    p->order_cap = 0;
    p->order_n_slabs = 0;
    if (has_order) {
        p->d_order = (uint32_t *)(base + o_order);
        p->order_cap = (uint32_t)slabs;
    }
    {
        std::vector<uint8_t> image(image_bytes, 0);   // control words, check record and order header start as zeros
        memcpy(image.data() + o_vals, p->h_vals, sizeof(int32_t) * (size_t)total_vals);
        if (n_scen) {
            memcpy(image.data() + o_scen, workload->scen_P, sizeof(int32_t) * n_scen);
            memcpy(image.data() + o_scen + sizeof(int32_t) * n_scen, workload->scen_O, sizeof(int32_t) * n_scen);
        }
        pf::sim_tables_place(p, base + o_sim, image.data() + o_sim);
        const cudaError_t e = cudaMemcpy(base, image.data(), image_bytes, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            pf::set_cuda_error(e, "pf_plan_create: upload");
            pf_plan_destroy(p);
            return PF_ECUDA;
        }
    }
    if (phase == PF_PHASE_TRAIN) {
        const cudaError_t e = pf::streams_acquire(p);
        if (e != cudaSuccess) {
            pf::set_cuda_error(e, "pf_plan_create: side stream");
            pf_plan_destroy(p);
            return PF_ECUDA;
        }
    }
    *out = p;
    return PF_OK;
}

extern "C" int pf_timing_enable(pf_plan_t *p, int on)
{
    if (!p) return PF_EINVAL;
    if (!p->timing) p->timing = new pf::Timing;
    ((pf::Timing *)p->timing)->on = on != 0;
    return PF_OK;
}

extern "C" int pf_timing_classes(pf_plan_t *p, uint32_t mask, uint32_t every)
{
    if (!p) return PF_EINVAL;
    if (!p->timing) p->timing = new pf::Timing;
    pf::Timing *t = (pf::Timing *)p->timing;
    t->mask = mask;
    t->every = every ? every : 1;
    for (uint32_t &s : t->seen) s = 0;
    return PF_OK;
}

extern "C" int pf_timing_read(pf_plan_t *p, float *ms, uint32_t *kernels)
{
    if (!p || !ms || !kernels) return PF_EINVAL;
    for (int i = 0; i < PF_T_CLASSES; i++) ms[i] = 0.f, kernels[i] = 0;
    pf::Timing *t = (pf::Timing *)p->timing;
    if (!t) return PF_OK;
    for (auto &r : t->recs) {
        float x = 0.f;
        if (r.open) {   // never closed (an error return in between): no interval to report
            t->pool.push_back(r.a);
            t->pool.push_back(r.b);
            continue;
        }
        PF_CUDA_TRY(cudaEventSynchronize(r.b), "pf_timing_read");
        PF_CUDA_TRY(cudaEventElapsedTime(&x, r.a, r.b), "pf_timing_read");
        ms[r.cls] += x;
        kernels[r.cls] += (uint32_t)r.n_kernels;
        t->pool.push_back(r.a);
        t->pool.push_back(r.b);
    }
    t->recs.clear();
    return PF_OK;
}

// The checks' own check: one thread asks for element 7 of a 4-element array through PF_AT.  In the checked build the
// index comes back as 0 (the store lands inside the array) and the record names the site, index and length.
__global__ void check_selftest_kernel(unsigned int *chk, unsigned int *four_words)
{
    four_words[PF_AT(chk, 3 + 4 * (int)(threadIdx.x + 1), 4, pf::PF_SITE_TOPK_BUF) & 3] = 1u;
}

extern "C" int pf_check_selftest(pf_plan_t *p)
{
    if (!p) return PF_EINVAL;
#ifndef PF_BOUNDS_CHECK
    return PF_EUNSUPPORTED;
#else
    if (int rc_dev = pf::check_device(p)) return rc_dev;
    check_selftest_kernel<<<1, 1>>>(p->d_check, p->d_check + 8);   // words 8..11 of the record's block: scratch
    PF_CUDA_TRY(cudaGetLastError(), "pf_check_selftest");
    return PF_OK;
#endif
}

extern "C" int pf_check_read(pf_plan_t *p, uint32_t *out)
{
    if (!p || !out) return PF_EINVAL;
#ifndef PF_BOUNDS_CHECK
    for (int i = 0; i < 6; i++) out[i] = 0;
    return PF_EUNSUPPORTED;   // this build carries no index checks
#else
    if (int rc_dev = pf::check_device(p)) return rc_dev;
    PF_CUDA_TRY(cudaDeviceSynchronize(), "pf_check_read");
    PF_CUDA_TRY(cudaMemcpy(out, p->d_check, 6 * sizeof(uint32_t), cudaMemcpyDeviceToHost), "pf_check_read");
    PF_CUDA_TRY(cudaMemset(p->d_check, 0, 64), "pf_check_read");
    return PF_OK;
#endif
}

extern "C" int pf_bench_fill_span(pf_plan_t *p, uint64_t *n_blocks, uint64_t *block_candidates, uint64_t *scored_blocks,
                                  uint64_t *filled_blocks)
{
    if (!p || !n_blocks || !block_candidates || !scored_blocks || !filled_blocks || !p->d_order) return PF_EINVAL;
    if (int rc_dev = pf::check_device(p)) return rc_dev;
    uint32_t hdr[8] = {0};
    PF_CUDA_TRY(cudaDeviceSynchronize(), "pf_bench_fill_span");
    PF_CUDA_TRY(cudaMemcpy(hdr, p->d_order, sizeof(hdr), cudaMemcpyDeviceToHost), "pf_bench_fill_span");
    *n_blocks = hdr[2];
    *block_candidates = p->dev.slab;
    *scored_blocks = hdr[4];
    uint32_t ctl[4] = {0};
    PF_CUDA_TRY(cudaMemcpy(ctl, p->d_fill_ctl, sizeof(ctl), cudaMemcpyDeviceToHost), "pf_bench_fill_span");
    *filled_blocks = ctl[2];
    return PF_OK;
}

extern "C" void pf_plan_destroy(pf_plan_t *p)
{
    if (!p) return;
    if (p->timing) {
        pf::Timing *t = (pf::Timing *)p->timing;
        for (auto &r : t->recs) {
            cudaEventDestroy(r.a);
            cudaEventDestroy(r.b);
        }
        for (auto e : t->pool) cudaEventDestroy(e);
        delete t;
    }
    pf::free_sim_tables(p);
    // The device block and the streams go back to their caches.  Work of this plan may still be in flight on a stream
    // of the caller's; freeing the block would have waited for the device, so this does too.
    if (p->arena || p->side_stream) {
        int cur = -1;
        const bool switched = cudaGetDevice(&cur) == cudaSuccess && cur != p->device && cudaSetDevice(p->device) == cudaSuccess;
        cudaDeviceSynchronize();
        if (switched) cudaSetDevice(cur);
    }
    pf::streams_release(p);
    pf::arena_release(p->device, p->arena, p->arena_cap);
    free(p->h_vals);
    delete p;
}

extern "C" uint64_t pf_plan_size(const pf_plan_t *p) { return p ? p->size : 0; }

extern "C" int pf_decode(const pf_plan_t *p, uint64_t idx, pf_tuple_t *out)
{
    if (!p || !out) return PF_EINVAL;
    if (idx >= p->size) return PF_ERANGE;
    int32_t v[PF_MAX_AXES] = {0};
    uint64_t rem = idx;
    for (int a = 0; a < p->dev.n_axes; a++) {
        uint64_t r = p->dev.radix[a];
        v[a] = p->h_vals[p->dev.val_off[a] + (int)(rem % r)];
        rem /= r;
    }
    memset(out, 0, sizeof(*out));
    if (p->dev.phase == PF_PHASE_TRAIN) {
        out->kv = v[0]; out->rec = v[1]; out->sched = v[2]; out->mb = v[3]; out->v = v[4];
        out->ep = v[5]; out->pp = v[6]; out->tp = v[7]; out->dp = v[8]; out->world = v[9];
        out->shard = p->dev.n_axes > 10 ? v[10] : PF_SHARD_ZERO1;
    } else {
        out->kv = v[0]; out->chunk = v[1]; out->batch = v[2]; out->dpa = v[3];
        out->ep = v[4]; out->tp = v[5]; out->scen = v[6];
    }
    return PF_OK;
}
