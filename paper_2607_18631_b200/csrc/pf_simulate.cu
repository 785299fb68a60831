// pf_simulate.cu -- simulator tier: one warp per survivor, one lane per pipeline rank (Sec. 3.2: the
// list-scheduling timeline refines the schedules the closed form only approximates).
//
// Each lane walks its rank's fixed op order (1F1B and interleaved orders are generated on the fly from
// counters; the DualPipe-style order comes from a host-built table) and computes
//   end(op) = max(end of the rank's previous op, end(dependency) + latency) + duration.
// A forward of stage q needs the forward of stage q-1 of the same microbatch, a backward of stage q needs
// the backward of stage q+1; the op's own forward is already behind the lane's clock.  Within one stage,
// forwards (and backwards) finish in microbatch order, so "is the dependency done" is a per-stage counter
// compare and the end-time arrays in shared memory never need clearing.  Lanes advance in lock step with
// __syncwarp between rounds; a round in which no lane advances ends the candidate with PF_SIM_STALL, so
// the loop is bounded by the op count.
#include <cstdlib>
#include <cstring>
#include <vector>

#include "pf_eval.cuh"

namespace pf {

constexpr int kSimMaxWarps = 16;        // warps per block at most (each simulates one candidate at a time)

// DualPipe-style order tables: for every (pp, m) in the domain a byte string per rank,
// op = (j << 2) | (dir << 1) | is_backward, 2*m ops per rank.
struct SimTables {
    uint8_t *d_ops;                 // device copy of all tables
    int32_t *d_offset;              // [33][33]: offset of table (pp, m/2), -1 if absent
    std::vector<int32_t> h_offset;
    size_t bytes;
};

// Host: nominal list scheduling that DEFINES the DualPipe-style order (F = 1 tick, B = 2 ticks, zero
// latency).  At every event time each idle rank starts the ready op with the smallest
// (ready time, backward before forward, microbatch, direction); a forward at position q may start only
// while fewer than pp - q microbatches of its direction are in flight on the rank.  Within one
// (rank, direction, F/B) stream ops become ready in microbatch order, so only the four stream heads of a
// rank compete.
static bool build_dualpipe_table(int pp, int m, uint8_t *out /* [pp][2m] */)
{
    const int n = m / 2;
    // done_at[type][dir][q][j]: nominal completion tick, -1 while not started
    std::vector<int> done_at((size_t)4 * pp * n, -1);
    auto at = [&](int b, int d, int q, int j) -> int & { return done_at[(((size_t)b * 2 + d) * pp + q) * n + j]; };
    std::vector<int> head((size_t)pp * 4, 0);  // next microbatch per (rank, dir, type)
    std::vector<int> live((size_t)pp * 2, 0), free_at(pp, 0), len(pp, 0);
    int remaining = 4 * pp * n, now = 0;
    while (remaining > 0) {
        for (int r = 0; r < pp; r++) {
            if (free_at[r] > now) continue;
            int best_b = -1, best_d = 0, best_j = 0, best_q = 0, best_ready = 0;
            for (int d = 0; d < 2; d++) {
                const int q = d ? pp - 1 - r : r;
                for (int b = 1; b >= 0; b--) {
                    const int j = head[(r * 2 + d) * 2 + b];
                    if (j >= n) continue;
                    int ready = 0;
                    if (b == 0) {
                        if (q > 0) {
                            int e = at(0, d, q - 1, j);
                            if (e < 0 || e > now) continue;
                            ready = e;
                        }
                        if (live[r * 2 + d] >= pp - q) continue;
                    } else {
                        int e = at(0, d, q, j);
                        if (e < 0 || e > now) continue;
                        ready = e;
                        if (q < pp - 1) {
                            int e2 = at(1, d, q + 1, j);
                            if (e2 < 0 || e2 > now) continue;
                            ready = e2 > ready ? e2 : ready;
                        }
                    }
                    bool better;
                    if (best_b < 0) better = true;
                    else if (ready != best_ready) better = ready < best_ready;
                    else if (b != best_b) better = b > best_b;
                    else if (j != best_j) better = j < best_j;
                    else better = d < best_d;
                    if (better) best_b = b, best_d = d, best_j = j, best_q = q, best_ready = ready;
                }
            }
            if (best_b < 0) continue;
            const int fin = now + (best_b ? 2 : 1);
            at(best_b, best_d, best_q, best_j) = fin;
            free_at[r] = fin;
            head[(r * 2 + best_d) * 2 + best_b]++;
            live[r * 2 + best_d] += best_b ? -1 : 1;
            out[(size_t)r * 2 * m + len[r]++] = (uint8_t)((best_j << 2) | (best_d << 1) | best_b);
            remaining--;
        }
        int next = -1;
        for (int r = 0; r < pp; r++)
            if (free_at[r] > now && (next < 0 || free_at[r] < next)) next = free_at[r];
        if (next < 0) return remaining == 0;  // nothing running and nothing ready: would never finish
        now = next;
    }
    return true;
}

// Called once by pf_plan_create for training plans: builds and uploads the order tables.
int build_sim_tables(pf_plan_t *p)
{
    if (p->sim_tables) return PF_OK;
    SimTables *t = new SimTables;
    t->d_ops = nullptr;
    t->d_offset = nullptr;
    t->h_offset.assign(33 * 33, -1);
    std::vector<uint8_t> ops;
    // only if a DualPipe-class schedule can pass the dry-run rules (mapped, or unconstrained mode);
    // depths from the pp axis (1 or even, <= 32)
    bool any_dual = false;
    for (int s = 0; s < p->dev.n_sched; s++)
        any_dual |= p->dev.sched[s].kind == PF_KIND_DUALPIPE && (p->dev.sched[s].mapped || !p->dev.enforce);
    if (any_dual && p->dev.phase == PF_PHASE_TRAIN) {
        const int32_t *pps = p->h_vals + p->dev.val_off[6];
        for (int i = 0; i < p->axis_len[6]; i++) {
            const int pp = pps[i];
            if (pp > PF_SIM_MAX_RANKS || (pp > 1 && (pp & 1))) continue;
            if (t->h_offset[pp * 33 + 1] >= 0) continue;
            for (int n = 1; n <= PF_SIM_WINDOW / 2; n++) {
                const int m = 2 * n;
                size_t off = ops.size();
                ops.resize(off + (size_t)pp * 2 * m);
                if (!build_dualpipe_table(pp, m, ops.data() + off)) {
                    delete t;
                    return PF_EINVAL;
                }
                t->h_offset[pp * 33 + n] = (int32_t)off;
            }
        }
    }
    t->bytes = ops.size();
    cudaError_t e = cudaMalloc((void **)&t->d_offset, sizeof(int32_t) * 33 * 33);
    if (e == cudaSuccess)
        e = cudaMemcpy(t->d_offset, t->h_offset.data(), sizeof(int32_t) * 33 * 33, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMalloc((void **)&t->d_ops, ops.size() ? ops.size() : 16);
    if (e == cudaSuccess && !ops.empty()) e = cudaMemcpy(t->d_ops, ops.data(), ops.size(), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        set_cuda_error(e, "simulator tables");
        if (t->d_offset) cudaFree(t->d_offset);
        if (t->d_ops) cudaFree(t->d_ops);
        delete t;
        return PF_ECUDA;
    }
    p->sim_tables = t;
    return PF_OK;
}

void free_sim_tables(pf_plan_t *p)
{
    SimTables *t = (SimTables *)p->sim_tables;
    if (!t) return;
    if (t->d_offset) cudaFree(t->d_offset);
    if (t->d_ops) cudaFree(t->d_ops);
    delete t;
    p->sim_tables = nullptr;
}

// ------------------------------------------------------------------ device

__device__ __forceinline__ uint32_t mix32(uint32_t x)
{
    x ^= x >> 16;
    x *= 0x7feb352du;
    x ^= x >> 15;
    x *= 0x846ca68bu;
    x ^= x >> 16;
    return x;
}

// multiplicative jitter in [0.9, 1.1): counter hash of (seed, candidate, stage, F/B)
__device__ __forceinline__ float jitter(uint32_t seed_mixed, uint64_t idx, int q, int is_b)
{
    uint32_t h = mix32(seed_mixed ^ (uint32_t)idx);
    h = mix32(h ^ (uint32_t)(idx >> 32));
    h = mix32(h ^ (uint32_t)(2 * q + is_b));
    float u = (float)(h >> 8) * (1.0f / 16777216.0f);
    return 0.9f + 0.2f * u;
}

constexpr int kSimClasses = 7;          // timeline sizes 256 << c entries (stage streams x microbatches)
__host__ __device__ inline int sim_class_entries(int c) { return 256 << c; }

struct SimArgs {
    const uint64_t *surv;
    uint64_t n;
    const uint64_t *d_n;            // optional device-side count
    uint32_t seed;
    float *tput_sim;
    uint8_t *status;
    unsigned int *work;             // [kSimClasses] work-queue heads, zeroed before launch
    unsigned int *cls_count;        // [kSimClasses] list lengths, zeroed before the classify kernel
    uint32_t *cls_list;             // [kSimClasses][n] positions in surv, grouped by timeline size
    const int32_t *vals;
    const uint8_t *dual_ops;
    const int32_t *dual_off;
    int q_max;                      // stages per candidate at most (plan-wide)
    int cls_hi;                     // largest class the plan can produce
    int pool_floats;                // dynamic shared memory of a block, in floats
};

// Pre-pass: one thread per survivor computes how many timeline entries its simulation needs and files the
// survivor under the smallest class that holds them, so each class can run with as many warps per SM as its
// shared-memory footprint allows.  Entries that cannot be simulated (outside the domain, malformed) go to
// class 0, where the simulator kernel rejects them before touching the timeline.
template <typename RI>
__global__ void __launch_bounds__(256) sim_classify_kernel(const __grid_constant__ DevPlan P, const SimArgs A)
{
    uint64_t n = A.n;
    if (A.d_n) {
        uint64_t dn = *A.d_n;
        n = dn < n ? dn : n;
    }
    const uint64_t w = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int cls = -1;
    if (w < n) {
        uint64_t rem = A.surv[w];
        int v[PF_MAX_AXES];
#pragma unroll
        for (int a = 0; a < PF_MAX_AXES; a++) {
            uint64_t r = P.radix[a];
            uint64_t q = rem / r;
            v[a] = __ldg(A.vals + P.val_off[a] + (int)(rem - q * r));
            rem = q;
        }
        const int s = v[2], mb = v[3], vv = v[4], pp = v[6], tp = v[7];
        RI dp = (RI)v[8];
        if (v[8] == 0) dp = (RI)v[9] / ((RI)tp * (RI)pp);
        const int kind = P.sched[s].kind;
        const int v_eff = vv == 0 ? (kind == PF_KIND_INTERLEAVED ? 2 : 1) : vv;
        cls = 0;
        const RI dpmb = dp * (RI)mb;
        if (dpmb != 0 && pp <= PF_SIM_MAX_RANKS && v_eff <= PF_SIM_MAX_V) {
            RI m = (RI)P.gbs / dpmb;
            int m_sim = m < (RI)PF_SIM_WINDOW ? (int)m : PF_SIM_WINDOW;
            if (kind == PF_KIND_INTERLEAVED) m_sim = (m_sim / pp) * pp;
            const int streams = kind == PF_KIND_DUALPIPE ? pp : pp * v_eff;  // DualPipe: 2 directions x m/2
            const int entries = streams * m_sim;
            while (cls < kSimClasses - 1 && sim_class_entries(cls) < entries) cls++;
            if (sim_class_entries(cls) < entries || streams > A.q_max) cls = 0;   // cannot be a feasible plan
        }
    }
    // warp-aggregated append per class
    for (int c = 0; c < kSimClasses; c++) {
        const unsigned mask = __ballot_sync(0xFFFFFFFFu, cls == c);
        if (mask == 0) continue;
        const int lane = threadIdx.x & 31, leader = __ffs(mask) - 1;
        unsigned int base = 0;
        if (lane == leader) base = atomicAdd(A.cls_count + c, (unsigned int)__popc(mask));
        base = __shfl_sync(0xFFFFFFFFu, base, leader);
        if (cls == c) A.cls_list[(size_t)c * A.n + base + __popc(mask & ((1u << lane) - 1u))] = (uint32_t)w;
    }
}

// per-warp shared memory of class c: endF[E], endB[E], durF[q_max], durB[q_max]
__host__ __device__ inline size_t sim_warp_floats(int entries, int q_max) { return (size_t)2 * entries + 2 * q_max; }

// The three round loops.  In every round a lane runs at most its next op, and only if the op it waits for
// has already published its end time; the body is branch-free apart from that test, so the lanes of a warp
// stay converged and a round costs one shared-memory poll plus one vote.  Every 64 rounds some lane must
// have advanced, otherwise the candidate is reported as stalled: the loops are bounded by the op count.
struct SimLane {
    float clock;
    bool stalled;
};

#define PF_SIM_ROUND_END()                                               \
    if (!__any_sync(0xFFFFFFFFu, done < total_ops)) break;               \
    if ((++rounds & 63) == 0) {                                          \
        if (!__any_sync(0xFFFFFFFFu, moved)) {                           \
            st.stalled = true;                                           \
            break;                                                       \
        }                                                                \
        moved = false;                                                   \
    }

// 1F1B: rank = stage = lane; `warm` forwards, then one forward / one backward, then the remaining backwards
__device__ __forceinline__ void sim_rounds_1f1b(volatile float *endF, volatile float *endB, const float *durF,
                                                const float *durB, int lane, int pp, int nj, int warm, int total_ops,
                                                float lat, SimLane &st)
{
    const bool depF = lane > 0, depB = lane < pp - 1;
    volatile float *inF = endF + (depF ? lane - 1 : lane) * nj, *inB = endB + (depB ? lane + 1 : lane) * nj;
    volatile float *outF = endF + lane * nj, *outB = endB + lane * nj;
    const float dF = lane < pp ? durF[lane] : 0.f, dB = lane < pp ? durB[lane] : 0.f;
    int nF = 0, nB = 0, done = 0, rounds = 0;
    bool moved = false;
    float clock = 0.f;
    for (;;) {
        if (done < total_ops) {
            const bool isb = !(nF < warm || (nF < nj && nF - warm == nB));
            const int j = isb ? nB : nF;
            const bool dep = isb ? depB : depF;
            const float e = (isb ? inB : inF)[j];
            if (!dep || e >= 0.f) {
                clock = fmaxf(clock, dep ? e + lat : 0.f) + (isb ? dB : dF);
                (isb ? outB : outF)[j] = clock;
                nF += isb ? 0 : 1;
                nB += isb ? 1 : 0;
                done++;
                moved = true;
            }
        }
        PF_SIM_ROUND_END()
    }
    st.clock = clock;
}

// Interleaved: v chunks per rank; unit k of a rank is microbatch (k / (pp v)) pp + k mod pp of chunk
// (k mod (pp v)) / pp, backward units walk the chunks downward; cursors advance without divisions
__device__ __forceinline__ void sim_rounds_interleaved(volatile float *endF, volatile float *endB, const float *durF,
                                                       const float *durB, int lane, int pp, int v, int nj, int U,
                                                       int warm, int total_ops, float lat, SimLane &st)
{
    const int Q = pp * v;
    int nF = 0, nB = 0, done = 0, rounds = 0;
    int fw = 0, fc = 0, fg = 0, bw = 0, bc = 0, bg = 0;
    bool moved = false;
    float clock = 0.f;
    for (;;) {
        if (done < total_ops) {
            const bool isb = !(nF < warm || (nF < U && nF - warm == nB));
            const int cw = isb ? bw : fw, cc = isb ? bc : fc, cg = isb ? bg : fg;
            const int j = cg * pp + cw;
            const int q = (isb ? v - 1 - cc : cc) * pp + lane;
            const bool dep = isb ? (q < Q - 1) : (q > 0);
            const int nb = dep ? (isb ? q + 1 : q - 1) : q;
            volatile float *arr = isb ? endB : endF;
            const float e = arr[nb * nj + j];
            const float dur = (isb ? durB : durF)[q];
            if (!dep || e >= 0.f) {
                clock = fmaxf(clock, dep ? e + lat : 0.f) + dur;
                arr[q * nj + j] = clock;
                int w_ = cw + 1, c_ = cc, g_ = cg;
                if (w_ == pp) {
                    w_ = 0;
                    if (++c_ == v) c_ = 0, g_++;
                }
                if (isb) bw = w_, bc = c_, bg = g_, nB++;
                else fw = w_, fc = c_, fg = g_, nF++;
                done++;
                moved = true;
            }
        }
        PF_SIM_ROUND_END()
    }
    st.clock = clock;
}

// DualPipe-style: two directions; the per-rank order comes from the host-built table
__device__ __forceinline__ void sim_rounds_dual(volatile float *endF, volatile float *endB, const float *durF,
                                                const float *durB, int lane, int pp, int nj, const uint8_t *ops,
                                                int total_ops, float lat, SimLane &st)
{
    int done = 0, rounds = 0;
    bool moved = false;
    float clock = 0.f;
    for (;;) {
        if (done < total_ops) {
            const uint32_t op = __ldg(ops + done);
            const bool isb = op & 1;
            const int d = (op >> 1) & 1, j = op >> 2;
            const int q = d ? pp - 1 - lane : lane;
            const int sidx = d * pp + q;
            const bool dep = isb ? (q < pp - 1) : (q > 0);
            const int nb = dep ? (isb ? sidx + 1 : sidx - 1) : sidx;
            volatile float *arr = isb ? endB : endF;
            const float e = arr[nb * nj + j];
            const float dur = (isb ? durB : durF)[q];
            if (!dep || e >= 0.f) {
                clock = fmaxf(clock, dep ? e + lat : 0.f) + dur;
                arr[sidx * nj + j] = clock;
                done++;
                moved = true;
            }
        }
        PF_SIM_ROUND_END()
    }
    st.clock = clock;
}
#undef PF_SIM_ROUND_END

// One launch serves every class.  A block owns a fixed pool of shared memory; while it works on class c as
// many of its warps as fit (pool / footprint) pull candidates from that class' queue, the others wait at the
// barrier that separates two classes.
template <typename RI>
__global__ void __launch_bounds__(kSimMaxWarps * 32) simulate_kernel(const __grid_constant__ DevPlan P, const SimArgs A)
{
    extern __shared__ float s_mem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t seed_mixed = mix32(A.seed + 0x9e3779b9u);

    // Blocks start on different classes (cyclic, staggered by block number) so that all classes are in
    // progress at once; a class whose queue is already drained is skipped, decided once per block.
    __shared__ int s_skip;
    const int n_classes = A.cls_hi + 1;
    for (int step = 0; step < n_classes; step++) {
    const int cls = (A.cls_hi - (int)(blockIdx.x % n_classes) - step + 2 * n_classes) % n_classes;
    const unsigned int n_cls = A.cls_count[cls];
    if (threadIdx.x == 0) s_skip = *reinterpret_cast<volatile unsigned int *>(A.work + cls) >= n_cls;
    __syncthreads();
    const bool skip = s_skip != 0;
    __syncthreads();
    if (skip) continue;
    const int E = sim_class_entries(cls);
    const int per_warp = (int)sim_warp_floats(E, A.q_max);
    const int active_warps = min((int)(blockDim.x >> 5), A.pool_floats / per_warp);
    if (warp < active_warps) {
    float *base = s_mem + (size_t)warp * per_warp;
    // End times are written by the lane that owns the stage and polled by its neighbour: one 32-bit word per
    // op, negative while the op has not finished, so a single volatile load answers "done, and when".
    volatile float *endF = base;
    volatile float *endB = base + E;
    float *durF = base + 2 * (size_t)E;
    float *durB = durF + A.q_max;
    const uint32_t *list = A.cls_list + (size_t)cls * A.n;

    for (;;) {
        unsigned int wi = 0;
        if (lane == 0) wi = atomicAdd(A.work + cls, 1u);
        wi = __shfl_sync(0xFFFFFFFFu, wi, 0);
        if (wi >= n_cls) break;
        const uint32_t w = list[wi];
        const uint64_t idx = A.surv[w];

        // ---- every lane re-derives the candidate (uniform across the warp)
        TrainTuple c;
        {
            int v[PF_MAX_AXES];
            uint64_t rem = idx;
#pragma unroll
            for (int a = 0; a < PF_MAX_AXES; a++) {
                uint64_t r = P.radix[a];
                uint64_t q = rem / r;
                v[a] = __ldg(A.vals + P.val_off[a] + (int)(rem - q * r));
                rem = q;
            }
            c.kv = v[0]; c.rec = v[1]; c.s = v[2]; c.mb = v[3]; c.v = v[4];
            c.ep = v[5]; c.pp = v[6]; c.tp = v[7]; c.dp = v[8]; c.world = v[9];
        }
        RI dp, world;
        TrainDerived<RI> D;
        TrainMem M;
        int reason = train_layout_rules<RI>(P, c, 1, 3, dp, world);
        if (reason == 0) reason = train_plan_rules<RI>(P, c, dp, world, 1, D);
        if (reason == 0) {
            train_memory<RI>(P, c, D, M);
            if (M.mem > P.budget_bytes) reason = PF_R_MEMORY;
        }
        if (reason != 0) {
            if (lane == 0) {
                if (A.tput_sim) A.tput_sim[w] = 0.f;
                if (A.status) A.status[w] = PF_SIM_UNSUPPORTED;
            }
            continue;
        }
        TrainTimes T;
        train_times<RI>(P, c, D, M, T);
        const int pp = c.pp, v = D.v_eff, kind = D.kind;
        if (pp > PF_SIM_MAX_RANKS || v > PF_SIM_MAX_V) {
            if (lane == 0) {
                if (A.tput_sim) A.tput_sim[w] = train_price<RI>(P, c, D, T, train_pipe_analytic<RI>(P, c, D, T));
                if (A.status) A.status[w] = PF_SIM_UNSUPPORTED;
            }
            continue;
        }
        const bool dual = kind == PF_KIND_DUALPIPE;
        const int Q = dual ? pp : pp * v;
        // simulated window
        const long long m = (long long)D.m;
        int m_sim = m < PF_SIM_WINDOW ? (int)m : PF_SIM_WINDOW;
        if (kind == PF_KIND_INTERLEAVED) m_sim = (m_sim / pp) * pp;
        const int nj = dual ? m_sim / 2 : m_sim;      // microbatches per stage stream
        const int n_entries = (dual ? 2 * Q : Q) * nj;
        bool stalled = n_entries > E || Q > A.q_max;  // filed under a class that cannot hold it: never for a
                                                      // feasible plan, reported instead of overrunning

        // ---- stage durations (balanced layer split, head on the last stage, jitter) and cleared timeline
        __syncwarp();
        if (!stalled) {
            const int L_lo = P.L / Q, L_rem = P.L - L_lo * Q;
            for (int q = lane; q < Q; q += 32) {
                const float nq = (float)(L_lo + (q < L_rem ? 1 : 0));
                const bool last = q == Q - 1;
                durF[q] = (nq * T.F_l + (last ? T.headF : 0.f)) * jitter(seed_mixed, idx, q, 0);
                durB[q] = (nq * T.B_l + (last ? P.bwd_factor * T.headF : 0.f)) * jitter(seed_mixed, idx, q, 1);
            }
            for (int i = lane; i < n_entries; i += 32) {
                endF[i] = -1.f;
                endB[i] = -1.f;
            }
        }
        __syncwarp();

        // ---- walk the rank's order
        const bool rank_active = lane < pp;
        const int U = dual ? 2 * nj : nj * (kind == PF_KIND_INTERLEAVED ? v : 1);  // forward units of this rank
        const uint8_t *dops = nullptr;
        if (dual && !stalled) {
            const int off = __ldg(A.dual_off + pp * 33 + nj);
            if (off < 0) stalled = true;  // no table for this shape: report instead of reading out of bounds
            else dops = A.dual_ops + off + (size_t)lane * 2 * m_sim;
        }
        const int total_ops = (rank_active && !stalled) ? 2 * U : 0;
        SimLane sl;
        sl.clock = 0.f;
        sl.stalled = stalled;
        if (!stalled) {
            if (kind == PF_KIND_1F1B)
                sim_rounds_1f1b(endF, endB, durF, durB, lane, pp, nj, min(pp - lane - 1, U), total_ops, T.p, sl);
            else if (kind == PF_KIND_INTERLEAVED)
                sim_rounds_interleaved(endF, endB, durF, durB, lane, pp, v, nj, U,
                                       min(2 * (pp - lane - 1) + (v - 1) * pp, U), total_ops, T.p, sl);
            else
                sim_rounds_dual(endF, endB, durF, durB, lane, pp, nj, dops, total_ops, T.p, sl);
        }
        stalled = sl.stalled;
        const float clock = sl.clock;

        // ---- makespan, steady-state extension beyond the window, pricing
        float work = 0.f;
        if (rank_active && !stalled) {
            if (dual) {
                work = 0.5f * (durF[lane] + durB[lane] + durF[pp - 1 - lane] + durB[pp - 1 - lane]);
            } else {
                const int vv = kind == PF_KIND_INTERLEAVED ? v : 1;
                for (int cc = 0; cc < vv; cc++) work += durF[cc * pp + lane] + durB[cc * pp + lane];
            }
        }
        float span = rank_active ? clock : 0.f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            span = fmaxf(span, __shfl_xor_sync(0xFFFFFFFFu, span, off));
            work = fmaxf(work, __shfl_xor_sync(0xFFFFFFFFu, work, off));
        }
        if (lane == 0) {
            float tput = 0.f;
            if (!stalled) {
                float T_pipe = span;
                if (m > m_sim) T_pipe += (float)(m - m_sim) * work;
                tput = train_price<RI>(P, c, D, T, T_pipe);
            }
            if (A.tput_sim) A.tput_sim[w] = tput;
            if (A.status) A.status[w] = stalled ? PF_SIM_STALL : PF_SIM_OK;
        }
        __syncwarp();
    }
    }  // active warps of this class
    __syncthreads();  // the next class lays the pool out differently
    }  // classes
}

// ------------------------------------------------------------------ top-k over a dense score array
// position in the list is the tie-break (equal to index order for lists from pf_select_survivors)

struct DenseTopkArgs {
    const float *score;
    uint64_t n;
    const uint64_t *d_n;
    uint32_t k;
    unsigned long long *keys;
    unsigned int *key_count;
};

__global__ void __launch_bounds__(kThreads) dense_topk_kernel(const DenseTopkArgs A)
{
    __shared__ unsigned long long s_buf[kTopkCap];
    __shared__ int s_count;
    __shared__ unsigned long long s_thr;
    __shared__ int s_base[2];
    const int tid = threadIdx.x;
    if (tid == 0) {
        s_count = 0;
        s_thr = 0ull;
    }
    __syncthreads();
    uint64_t n = A.n;
    if (A.d_n) {
        uint64_t dn = *A.d_n;
        n = dn < n ? dn : n;
    }
    int room = kTopkCap / kThreads;
    unsigned long long thr = 0ull;
    for (uint64_t base = (uint64_t)blockIdx.x * kThreads; base < n; base += (uint64_t)gridDim.x * kThreads) {
        if (room == 0) {
            __syncthreads();
            if (s_count > kTopkCap - kThreads) tk_prune<kTopkCap / 2 / kThreads>(s_buf, &s_count, &s_thr, (int)A.k);
            room = (kTopkCap - s_count) / kThreads;
            thr = s_thr;
            __syncthreads();
        }
        const uint64_t i = base + tid;
        const float s = i < n ? A.score[i] : 0.f;
        tk_push(s_buf, &s_count, thr, s > 0.f, make_key(s, (uint32_t)i));
        room--;
    }
    tk_prune<kTopkCap / 2 / kThreads>(s_buf, &s_count, &s_thr, (int)A.k);
    tk_flush(s_buf, s_count, 0ull, s_base, A.keys, A.key_count);
}

struct SimLayout {
    size_t off_ctrl, off_lists, off_scores, off_topk, total;
    int topk_blocks;
    uint64_t topk_keys_max;
    TopkLayout tk;
};

static SimLayout sim_layout(const pf_plan_t *p, uint64_t n, uint32_t k)
{
    SimLayout l;
    const size_t nn = (size_t)(n ? n : 1);
    l.off_ctrl = 0;                       // work[kSimClasses], cls_count[kSimClasses]
    l.off_lists = 256;
    l.off_scores = l.off_lists + (((size_t)kSimClasses * nn * 4 + 255) & ~(size_t)255);
    l.off_topk = l.off_scores + ((nn * 4 + 255) & ~(size_t)255);
    uint64_t tb = (n + kThreads - 1) / kThreads;
    uint64_t cap = (uint64_t)p->sm_count * 2;
    l.topk_blocks = (int)(tb < 1 ? 1 : (tb > cap ? cap : tb));
    l.topk_keys_max = (uint64_t)l.topk_blocks * (k ? k : 1);
    if (l.topk_keys_max > nn) l.topk_keys_max = nn < (k ? k : 1) ? (k ? k : 1) : nn;
    l.tk = topk_layout(l.topk_keys_max, k);
    l.total = l.off_topk + (k ? l.tk.total : 0);
    return l;
}

// plan-wide bound on stages per candidate inside the simulator's domain
static int plan_q_max(const pf_plan_t *p)
{
    int pp_max = 1, v_max = 1;
    const int32_t *pps = p->h_vals + p->dev.val_off[6];
    for (int i = 0; i < p->axis_len[6]; i++)
        if (pps[i] <= PF_SIM_MAX_RANKS && pps[i] > pp_max) pp_max = pps[i];
    const int32_t *vs = p->h_vals + p->dev.val_off[4];
    for (int i = 0; i < p->axis_len[4]; i++) {
        int v = vs[i] == 0 ? 2 : vs[i];
        if (v <= PF_SIM_MAX_V && v > v_max) v_max = v;
    }
    long long q = (long long)pp_max * v_max;
    if (q > p->dev.L) q = p->dev.L;  // the layer rule admits pp*v <= L only
    if (q < pp_max) q = pp_max;
    return (int)q;
}

template <typename RI>
static int launch_simulate(pf_plan_t *p, SimArgs a, uint64_t n, cudaStream_t st, int *n_kernels)
{
    *n_kernels = 0;
    sim_classify_kernel<RI><<<(unsigned int)((n + 255) / 256), 256, 0, st>>>(p->dev, a);
    count_launch();
    (*n_kernels)++;
    PF_CUDA_TRY(cudaGetLastError(), "sim_classify_kernel launch");
    // largest class the plan can produce, and a pool that holds at least one such timeline
    const int entries_max = a.q_max * PF_SIM_WINDOW;
    int cls_hi = 0;
    while (cls_hi < kSimClasses - 1 && sim_class_entries(cls_hi) < entries_max) cls_hi++;
    const size_t biggest = sim_warp_floats(sim_class_entries(cls_hi), a.q_max) * sizeof(float);
    if (biggest > 226 * 1024) return PF_EUNSUPPORTED;   // 227 KB per block minus the kernel's static words
    size_t pool = 72 * 1024;                         // three blocks per SM when the largest timeline allows
    if (pool < biggest) pool = biggest;
    int per_sm = (int)((size_t)(227 * 1024) / (pool + 1024));
    per_sm = per_sm < 1 ? 1 : per_sm;
    a.cls_hi = cls_hi;
    a.pool_floats = (int)(pool / sizeof(float));
    const uint64_t cap = (uint64_t)p->sm_count * per_sm;
    const int grid = (int)(n < cap ? n : cap);
    PF_CUDA_TRY(cudaFuncSetAttribute(simulate_kernel<RI>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pool),
                "simulate_kernel smem");
    simulate_kernel<RI><<<grid, kSimMaxWarps * 32, pool, st>>>(p->dev, a);
    count_launch();
    (*n_kernels)++;
    PF_CUDA_TRY(cudaGetLastError(), "simulate_kernel launch");
    return PF_OK;
}

}  // namespace pf

using namespace pf;

extern "C" int pf_dualpipe_order(int pp, int m, uint8_t *out_ops)
{
    if (!out_ops || pp < 1 || pp > PF_SIM_MAX_RANKS || (pp > 1 && (pp & 1)) || m < 2 || (m & 1) || m > PF_SIM_WINDOW)
        return PF_EINVAL;
    return build_dualpipe_table(pp, m, out_ops) ? PF_OK : PF_EINVAL;
}

extern "C" size_t pf_simulate_workspace(const pf_plan_t *p, uint64_t n, uint32_t k)
{
    if (!p) return 0;
    return sim_layout(p, n, k).total;
}

extern "C" int pf_simulate(pf_plan_t *p, const uint64_t *d_surv_idx, uint64_t n, const uint64_t *d_n,
                           uint32_t jitter_seed, float *d_tput_sim, uint8_t *d_sim_status, uint32_t k,
                           uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count, void *d_workspace,
                           size_t workspace_bytes, void *stream)
{
    if (!p || !d_surv_idx) return PF_EINVAL;
    if (p->dev.phase != PF_PHASE_TRAIN) return PF_EUNSUPPORTED;
    if (k > PF_K_MAX) return PF_EINVAL;
    if (k > 0 && (!d_topk_idx || !d_topk_score || !d_topk_count)) return PF_EINVAL;
    if (n >= PF_MAX_COUNT) return PF_ERANGE;
    const SimLayout lay = sim_layout(p, n, k);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < lay.total) return PF_EWORKSPACE;
    if (!p->sim_tables) return PF_EINVAL;
    int rc = PF_OK;
    const SimTables *tab = (const SimTables *)p->sim_tables;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)d_workspace;
    float *scores = d_tput_sim ? d_tput_sim : (float *)(ws + lay.off_scores);

    SimArgs a;
    a.surv = d_surv_idx; a.n = n; a.d_n = d_n; a.seed = jitter_seed;
    a.tput_sim = scores; a.status = d_sim_status;
    a.work = (unsigned int *)(ws + lay.off_ctrl);
    a.cls_count = a.work + kSimClasses;
    a.cls_list = (uint32_t *)(ws + lay.off_lists);
    a.vals = p->d_vals; a.dual_ops = tab->d_ops; a.dual_off = tab->d_offset;
    a.q_max = plan_q_max(p);
    a.cls_hi = 0;
    a.pool_floats = 0;
    PF_CUDA_TRY(cudaMemsetAsync(ws + lay.off_ctrl, 0, 256, st), "pf_simulate: counter reset");
    if (n > 0) {
        int nk = 0;
        timing_begin(p, PF_T_SIMULATE, st);
        rc = p->dev.wide ? launch_simulate<unsigned long long>(p, a, n, st, &nk)
                         : launch_simulate<uint32_t>(p, a, n, st, &nk);
        timing_end(p, PF_T_SIMULATE, nk, st);
        if (rc != PF_OK) return rc;
    }
    if (k > 0) {
        uint8_t *tws = ws + lay.off_topk;
        PF_CUDA_TRY(cudaMemsetAsync(tws + lay.tk.off_ctrl, 0, 256, st), "pf_simulate: top-k reset");
        DenseTopkArgs t;
        t.score = scores; t.n = n; t.d_n = d_n; t.k = k;
        t.keys = (unsigned long long *)(tws + lay.tk.off_keys_a);
        t.key_count = (unsigned int *)(tws + lay.tk.off_ctrl) + 1;
        timing_begin(p, PF_T_TOPK, st);
        dense_topk_kernel<<<lay.topk_blocks, kThreads, 0, st>>>(t);
        count_launch();
        PF_CUDA_TRY(cudaGetLastError(), "dense_topk_kernel launch");
        int nk = 0;
        rc = launch_topk_reduce(tws, lay.tk, lay.topk_keys_max, k, 0, d_surv_idx, d_topk_idx, d_topk_score,
                                d_topk_count, st, &nk);
        timing_end(p, PF_T_TOPK, nk + 1, st);
        return rc;
    }
    return PF_OK;
}
