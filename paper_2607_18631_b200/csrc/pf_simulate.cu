// pf_simulate.cu -- simulator tier: a group of lanes per survivor, one lane per pipeline rank (Sec. 3.2: the
// list-scheduling timeline refines the schedules the closed form only approximates).
//
// Each lane walks its rank's fixed op order (1F1B and interleaved orders are generated on the fly from
// cursors; the DualPipe-style order comes from a host-built table) and computes
//   end(op) = max(end of the rank's previous op, end(dependency) + latency) + duration.
// A forward of stage q needs the forward of stage q-1 of the same microbatch, a backward of stage q needs
// the backward of stage q+1; the op's own forward is already behind the lane's clock.
//
// Launch structure: a counting-sort pre-pass (classify, offsets, scatter) bins the survivors by
// (timeline size class, lane-group width 4/8/16/32, round loop), then ONE simulate_kernel grid serves all
// bins, largest timelines first (of the kernel's two instances, for small and for large calls, the one that
// matches the actual survivor count; the other, if launched, ends at once).  Every warp owns a slice of the block's shared memory and runs its own
// candidates there; the timeline is one signed 32-bit word per (stage stream, microbatch), microbatch-major (word
// j * streams + stream, so that the lanes of a group touch neighbouring words) -- 0 nothing finished, +t forward
// ended at t, -t backward ended at t -- written by its owner lane and polled by the neighbour.  In a large call
// (kSimRingMinSurvivors) interleaved schedules run on a ring of 2 pp microbatch slots per stage stream instead
// (tagged two-word slots), which lets more candidates share a warp, pipelines of depth <= 4 take four lanes, and
// timeline indices are XORed with a constant of the lane group so that the groups of a warp use different banks.
// No block barrier is used, and a warp whose lanes make no progress for 64 rounds reports its unfinished
// candidates as PF_SIM_STALL, so every loop is bounded by the op count.
#include <cstdlib>
#include <cstring>
#include <vector>

#include "pf_eval.cuh"

namespace pf {


// DualPipe-style order tables: for every (pp, m) in the domain a byte string per rank,
// op = (j << 2) | (dir << 1) | is_backward, 2*m ops per rank.
struct SimTables {
    uint8_t *d_ops;                 // device copy of all tables (inside the plan's device block)
    int32_t *d_offset;              // [33][33]: offset of table (pp, m/2), -1 if absent
    std::vector<int32_t> h_offset;
    std::vector<uint8_t> h_ops;     // host copy, until it has been placed in the plan's device block
    size_t bytes;
};
constexpr size_t kSimOffsetBytes = (sizeof(int32_t) * 33 * 33 + 255) & ~(size_t)255;

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

// Called once by pf_plan_create for training plans: builds the order tables on the host; sim_tables_place puts them
// into the plan's device block.
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
    t->h_ops.swap(ops);
    p->sim_tables = t;
    return PF_OK;
}

// bytes of the plan's device block the tables take (both parts 256-byte aligned)
size_t sim_tables_bytes(const pf_plan_t *p)
{
    const SimTables *t = (const SimTables *)p->sim_tables;
    if (!t) return 0;
    return kSimOffsetBytes + (((t->bytes ? t->bytes : 16) + 255) & ~(size_t)255);
}

// The tables live at `dev` in the plan's device block; their bytes are written to `image`, the host copy of that
// stretch, which the caller uploads with the rest of the block.
void sim_tables_place(pf_plan_t *p, uint8_t *dev, uint8_t *image)
{
    SimTables *t = (SimTables *)p->sim_tables;
    if (!t) return;
    t->d_offset = (int32_t *)dev;
    t->d_ops = dev + kSimOffsetBytes;
    memcpy(image, t->h_offset.data(), sizeof(int32_t) * 33 * 33);
    if (!t->h_ops.empty()) memcpy(image + kSimOffsetBytes, t->h_ops.data(), t->h_ops.size());
    std::vector<uint8_t>().swap(t->h_ops);
}

void free_sim_tables(pf_plan_t *p)
{
    SimTables *t = (SimTables *)p->sim_tables;
    if (!t) return;
    delete t;   // (the device copy is part of the plan's device block)
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

// multiplicative jitter in [0.9, 1.1): counter hash of (seed, candidate, stage, F/B); `cand_hash` is the part of
// the chain that depends on the seed and the candidate only
__device__ __forceinline__ float jitter(uint32_t cand_hash, int q, int is_b)
{
    const uint32_t h = mix32(cand_hash ^ (uint32_t)(2 * q + is_b));
    float u = (float)(h >> 8) * (1.0f / 16777216.0f);
    return 0.9f + 0.2f * u;
}

constexpr int kSimClasses = 7;          // timeline sizes 256 << c entries (stage streams x microbatches)
constexpr int kSimGroups = 4;           // lanes per candidate: 4, 8, 16 or 32 (pipeline depth rounded up)
constexpr int kSimKinds = 4;            // round loop of a batch: the three schedule classes, and the interleaved one
                                        // on a ring timeline (kSimKindRing)
constexpr int kSimKindRing = 3;
constexpr int kSimBins = kSimClasses * kSimGroups * kSimKinds;   // 112
constexpr int kSimTab = 128;            // queue tables: bins rounded up to four per lane
constexpr int kSimThreads = 128;        // 4 warps per block, each with its own shared-memory slice
__host__ __device__ inline int sim_class_entries(int c) { return 256 << c; }
__host__ __device__ inline int sim_group_lanes(int g) { return 4 << g; }
// (four-lane groups only in large calls, like ring timelines: see kSimRingMinSurvivors)
__host__ __device__ inline int sim_group_of(int pp, bool narrow) { return (pp <= 4 && narrow) ? 0 : (pp <= 8 ? 1 : (pp <= 16 ? 2 : 3)); }
// stages a lane group's duration tables must hold: the plan-wide bound, or what the group's ranks can carry
__host__ __device__ inline int sim_group_stages(int lanes, int q_max)
{
    const int by_ranks = lanes * PF_SIM_MAX_V;
    return by_ranks < q_max ? by_ranks : q_max;
}
// An interleaved schedule keeps few microbatches of a stage in flight, so its timeline can be a ring of W = 2 pp
// microbatch slots per stage stream (a multiple of the order's window of pp microbatches) instead of one word per
// microbatch; a slot is then two words, tag and time, so that a reader can tell the lap.  Worth it when that is at
// least a size class smaller AND the call is large: a ring step costs a few instructions more than a full-timeline
// step, which a call of few survivors (bound by its longest op chain, warps to spare) feels, whereas a large call is
// bound by how many candidates a warp instruction serves (12,905 survivors: 0.147 ms full, 0.170 ms ring; 1e6: 6.6 ms
// full, 5.0 ms ring).
__host__ __device__ inline int sim_ring_slots(int pp) { return 2 * pp; }
constexpr uint64_t kSimRingMinSurvivors = 32768;

// What the simulator kernel needs about one survivor, worked out once by the pre-pass (one thread per survivor)
// instead of by every lane of the group that simulates it: the per-layer times, the hand-over latency, the rest of
// the step, the pricing, the shape.  64 bytes, read with four 16-byte loads.
struct __align__(16) SimRec {
    float F_l, B_l, F_ld, B_ld;     // forward / backward time of a MoE layer and of a leading dense layer
    float headF, p, rest, denom;    // head forward, stage hand-over, step time beyond the pipeline, world x taxes
    uint32_t hash, w, meta, m;      // jitter hash of (seed, candidate); position in the caller's list; shape; microbatches
    uint32_t pad[4];
};
static_assert(sizeof(SimRec) == 64, "SimRec is read as four 16-byte words");
// meta: pp - 1 (5 bits) | v - 1 (3 bits) << 5 | kind (2 bits) << 8 | m_sim (7 bits) << 10 | ring timeline << 17
__device__ __forceinline__ uint32_t sim_meta(int pp, int v, int kind, int m_sim, bool ring)
{
    return (uint32_t)(pp - 1) | ((uint32_t)(v - 1) << 5) | ((uint32_t)kind << 8) | ((uint32_t)m_sim << 10) |
           ((uint32_t)(ring ? 1 : 0) << 17);
}

struct SimArgs {
    const uint64_t *surv;
    uint64_t n;
    const uint64_t *d_n;            // optional device-side count
    uint32_t seed;
    float *tput_sim;
    uint8_t *status;
    unsigned int *work;             // [1] the batch queue's head
    unsigned int *bin_count;        // [kSimBins] survivors per bin
    unsigned int *bin_off;          // [kSimBins + 1] start of each bin in the record array
    unsigned int *bin_fill;         // [kSimBins] scatter cursors
    unsigned int *bin_seq;          // [kSimTab] bins in the order the batch queue serves them
    unsigned int *batch_pre;        // [kSimTab + 1] batches before each position of that order; last = all batches
    uint8_t *bin_of;                // [n] bin of each survivor (0xFF: not simulated)
    SimRec *recs;                   // [n] records, grouped by bin
    const int32_t *vals;
    const uint8_t *dual_ops;
    const int32_t *dual_off;
    int q_max;                      // stages per candidate at most (plan-wide)
    int cls_hi;                     // largest class the plan can produce
    int warp_floats;                // shared-memory slice of one warp, in floats
};

// candidates a warp simulates side by side in one batch of a bin: as many lane groups as fit the warp, as many
// timelines as fit its slice
__host__ __device__ inline int sim_bin_batch(int bin, int cls_hi)
{
    const int cls = bin / (kSimGroups * kSimKinds), gi = (bin / kSimKinds) % kSimGroups;
    const int by_lanes = 32 / sim_group_lanes(gi), by_room = sim_class_entries(cls_hi) / sim_class_entries(cls);
    return by_lanes < by_room ? by_lanes : by_room;
}

// A survivor as the pre-pass sees it: decoded, checked, timed.
template <typename RI>
struct SimCand {
    TrainTuple c;
    TrainDerived<RI> D;
    TrainMem M;
    TrainTimes T;
    int reason;
};

template <typename RI>
__device__ __forceinline__ void sim_decode(const DevPlan &P, const int32_t *vals, uint64_t idx, SimCand<RI> &S,
                                           bool with_times)
{
    int v[PF_MAX_AXES];
    uint64_t rem = idx;
#pragma unroll
    for (int a = 0; a < PF_MAX_AXES; a++) {
        uint64_t r = P.radix[a];
        uint64_t q = rem / r;
        v[a] = __ldg(vals + P.val_off[a] + (int)(rem - q * r));
        rem = q;
    }
    TrainTuple &c = S.c;
    c.kv = v[0]; c.rec = v[1]; c.s = v[2]; c.mb = v[3]; c.v = v[4];
    c.ep = v[5]; c.pp = v[6]; c.tp = v[7]; c.dp = v[8]; c.world = v[9];
    c.sh = P.n_axes > 10 ? v[10] : PF_SHARD_ZERO1;
    RI dp, world;
    S.reason = train_layout_rules<RI>(P, c, 1, 3, dp, world);
    if (S.reason == 0) S.reason = train_plan_rules<RI>(P, c, dp, world, 1, S.D);
    if (S.reason == 0) {
        train_memory<RI>(P, c, S.D, S.M);
        if (S.M.mem > P.budget_bytes) S.reason = PF_R_MEMORY;
    }
    if (S.reason == 0 && with_times) train_times<RI>(P, c, S.D, S.M, S.T);
}

// timeline shape of a feasible candidate inside the simulator's domain
template <typename RI>
__device__ __forceinline__ void sim_shape(const SimCand<RI> &S, int &m_sim, int &streams)
{
    const int pp = S.c.pp, kind = S.D.kind;
    m_sim = S.D.m < (RI)PF_SIM_WINDOW ? (int)S.D.m : PF_SIM_WINDOW;
    if (kind == PF_KIND_INTERLEAVED) m_sim = (m_sim / pp) * pp;
    streams = kind == PF_KIND_DUALPIPE ? pp : pp * S.D.v_eff;   // DualPipe-style: 2 directions x m/2
}
// timeline words of a shape and whether it goes on a ring (interleaved schedules only; see sim_ring_slots)
__device__ __forceinline__ int sim_entries(int kind, int pp, int streams, int m_sim, uint64_t n_call, bool &ring)
{
    const int full = streams * m_sim;
    ring = false;
    if (kind != PF_KIND_INTERLEAVED || m_sim <= sim_ring_slots(pp) || n_call < kSimRingMinSurvivors) return full;
    const int on_ring = streams * sim_ring_slots(pp) * 2;
    int c_full = 0, c_ring = 0;
    while (c_full < kSimClasses - 1 && sim_class_entries(c_full) < full) c_full++;
    while (c_ring < kSimClasses - 1 && sim_class_entries(c_ring) < on_ring) c_ring++;
    ring = c_ring < c_full;
    return ring ? on_ring : full;
}

// Pre-pass 1, one thread per survivor: decode it, run the predicate again (the list may hold anything), and
//   - infeasible: score 0, status UNSUPPORTED, written here;
//   - feasible but outside the simulator's domain (or a shape no bin holds): the analytic score, status
//     UNSUPPORTED, written here;
//   - otherwise its bin: the smallest timeline class that holds its stage streams x microbatches, the lane-group
//     width that holds its pipeline depth, its schedule class -- so that timelines of similar size are scheduled
//     together, several shallow pipelines share a warp and a batch runs one specialised loop.
template <typename RI>
__global__ void __launch_bounds__(256) sim_classify_kernel(const __grid_constant__ DevPlan P, const SimArgs A)
{
    chain_enter();
    uint64_t n = A.n;
    if (A.d_n) {
        uint64_t dn = *A.d_n;
        n = dn < n ? dn : n;
    }
    const uint64_t w = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int bin = -1;
    if (w < n) {
        SimCand<RI> S;
        sim_decode<RI>(P, A.vals, A.surv[w], S, false);
        float out = 0.f;
        bool direct = true;
        if (S.reason == 0) {
            int m_sim, streams;
            sim_shape<RI>(S, m_sim, streams);
            const int pp = S.c.pp;
            bool ring;
            const int entries = sim_entries(S.D.kind, pp, streams, m_sim, n, ring);
            int cls = 0;
            while (cls < kSimClasses - 1 && sim_class_entries(cls) < entries) cls++;
            const bool table_ok = S.D.kind != PF_KIND_DUALPIPE || __ldg(A.dual_off + pp * 33 + m_sim / 2) >= 0;
            if (pp <= PF_SIM_MAX_RANKS && S.D.v_eff <= PF_SIM_MAX_V && cls <= A.cls_hi &&
                sim_class_entries(cls) >= entries && streams <= A.q_max &&
                streams <= sim_group_stages(sim_group_lanes(sim_group_of(pp, n >= kSimRingMinSurvivors)), A.q_max) && table_ok) {
                bin = (cls * kSimGroups + sim_group_of(pp, n >= kSimRingMinSurvivors)) * kSimKinds + (ring ? kSimKindRing : S.D.kind);
                direct = false;
            } else {
                train_times<RI>(P, S.c, S.D, S.M, S.T);
                out = train_price<RI>(P, S.c, S.D, S.T, train_pipe_analytic<RI>(P, S.c, S.D, S.T));
                // inside the domain but without a bin (a shape the plan's bounds do not cover): reported, not run
                if (pp <= PF_SIM_MAX_RANKS && S.D.v_eff <= PF_SIM_MAX_V) out = 0.f;
            }
        }
        if (direct) {
            const bool in_domain = S.reason == 0 && S.c.pp <= PF_SIM_MAX_RANKS && S.D.v_eff <= PF_SIM_MAX_V;
            if (A.tput_sim) A.tput_sim[w] = out;
            if (A.status) A.status[w] = (uint8_t)(in_domain ? PF_SIM_STALL : PF_SIM_UNSUPPORTED);
        }
        A.bin_of[w] = (uint8_t)(bin < 0 ? 0xFF : bin);
    }
    // warp-aggregated count per bin
    const unsigned peers = __match_any_sync(0xFFFFFFFFu, bin);
    if (bin >= 0 && (int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(A.bin_count + bin, (unsigned int)__popc(peers));
}

// Pre-pass 2 (one warp): where each bin's records start, and the batch queue: bins are served interleaved
// schedules first, then DualPipe-style, then 1F1B (the per-rank op chains of an interleaved schedule are v times
// longer, so the longest simulations start first and the kernel's tail is short), larger timelines first within a
// class; batches are numbered through in that order.  Lane l owns bins / queue positions l, l + 32, l + 64 and
// l + 96, so every global word is read once, all loads in flight together.
__device__ __forceinline__ unsigned int warp_incl_scan(unsigned int x, int lane)
{
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned int y = __shfl_up_sync(0xFFFFFFFFu, x, off);
        if (lane >= off) x += y;
    }
    return x;
}
__global__ void __launch_bounds__(32) sim_offsets_kernel(const SimArgs A)
{
    chain_enter();
    constexpr int kQ = kSimTab / 32;   // table entries per lane: lane l owns entries l, l + 32, ...
    const int lane = threadIdx.x;
    unsigned int cnt[kQ], incl[kQ];
    unsigned int carry = 0;
#pragma unroll
    for (int h = 0; h < kQ; h++) {
        const int b = lane + 32 * h;
        cnt[h] = b < kSimBins ? A.bin_count[b] : 0u;
    }
#pragma unroll
    for (int h = 0; h < kQ; h++) {
        incl[h] = warp_incl_scan(cnt[h], lane);
        A.bin_off[lane + 32 * h] = carry + incl[h] - cnt[h];     // entries kSimBins .. kSimTab - 1 = all records
        carry += __shfl_sync(0xFFFFFFFFu, incl[h], 31);
    }
    // queue order: interleaved schedules on full timelines, on ring timelines, DualPipe-style, 1F1B; larger
    // timelines first within each; position -> bin
    unsigned int nb[kQ];
    int bin_at[kQ];
#pragma unroll
    for (int h = 0; h < kQ; h++) {
        const int pos = lane + 32 * h;
        const bool valid = pos < kSimBins;
        const int ko = pos / (kSimClasses * kSimGroups), rem = pos - ko * (kSimClasses * kSimGroups);
        const int cls = kSimClasses - 1 - rem / kSimGroups, gi = rem % kSimGroups;
        const int kind = ko == 0 ? PF_KIND_INTERLEAVED : ko == 1 ? kSimKindRing : ko == 2 ? PF_KIND_DUALPIPE : PF_KIND_1F1B;
        const int bin = valid ? (cls * kSimGroups + gi) * kSimKinds + kind : 0;
        unsigned int c = 0;
#pragma unroll
        for (int hh = 0; hh < kQ; hh++) {
            const unsigned int from = __shfl_sync(0xFFFFFFFFu, cnt[hh], bin & 31);
            if ((bin >> 5) == hh) c = from;
        }
        bin_at[h] = bin;
        nb[h] = 0u;
        if (valid && cls <= A.cls_hi) {
            const unsigned int per = (unsigned int)sim_bin_batch(bin, A.cls_hi);
            nb[h] = (c + per - 1) / per;
        }
    }
    carry = 0;
#pragma unroll
    for (int h = 0; h < kQ; h++) {
        const unsigned int b_incl = warp_incl_scan(nb[h], lane);
        A.bin_seq[lane + 32 * h] = (unsigned int)bin_at[h];
        A.batch_pre[lane + 32 * h] = carry + b_incl - nb[h];
        carry += __shfl_sync(0xFFFFFFFFu, b_incl, 31);
    }
    if (lane == 31) A.batch_pre[kSimTab] = carry;   // all batches
}

// Pre-pass 3, one thread per survivor again: the binned ones get their record -- every term the simulator kernel
// needs -- written at their place in the bin.
template <typename RI>
__global__ void __launch_bounds__(256) sim_records_kernel(const __grid_constant__ DevPlan P, const SimArgs A)
{
    chain_enter();
    uint64_t n = A.n;
    if (A.d_n) {
        uint64_t dn = *A.d_n;
        n = dn < n ? dn : n;
    }
    const uint64_t w = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int bin = (w < n && A.bin_of[w] != 0xFF) ? (int)A.bin_of[w] : -1;
    const unsigned peers = __match_any_sync(0xFFFFFFFFu, bin);
    const int lane = threadIdx.x & 31, leader = __ffs(peers) - 1;
    unsigned int base = 0;
    if (bin >= 0 && lane == leader) base = atomicAdd(A.bin_fill + bin, (unsigned int)__popc(peers));
    base = __shfl_sync(0xFFFFFFFFu, base, leader);
    if (bin < 0) return;
    const uint64_t idx = A.surv[w];
    SimCand<RI> S;
    sim_decode<RI>(P, A.vals, idx, S, true);
    const TrainTuple &c = S.c;
    TrainTimes &T = S.T;
    const DevSched &sc = P.sched[c.s];
    if (S.D.ov && sc.n_chunks > 0 && c.sh != PF_SHARD_ZERO1_OFFLOAD) {
        // the schedule says how it overlaps: the exposed communication of a MoE layer comes from its two-stream
        // timeline instead of the alpha-table's hidden fraction
        const float slow = fdiv(1.f, 1.f - sc.sm_frac), half = 0.5f * T.a2a;
        const float cF = T.cD + T.cE, cBt = P.bwd_factor * cF + T.rc;
        const float share = fdiv(T.cE, cF);
        const float fwd = two_stream_layer(T.cD * slow, T.cE * slow, half, half, sc.n_chunks);
        const float bwd = two_stream_layer(cBt * (1.f - share) * slow, cBt * share * slow, half, half, sc.n_chunks);
        T.F_l = T.tpc + fwd;
        T.B_l = T.tpc + bwd + (c.rec == PF_REC_FULL ? T.tpc + (fwd - cF * slow) : 0.f);
    }
    int m_sim, streams;
    sim_shape<RI>(S, m_sim, streams);
    bool ring;
    (void)sim_entries(S.D.kind, c.pp, streams, m_sim, n, ring);
    SimRec r;
    r.F_l = T.F_l; r.B_l = T.B_l; r.F_ld = T.F_ld; r.B_ld = T.B_ld;
    r.headF = T.headF; r.p = T.p;
    r.rest = (1.f - P.dp_overlap_frac) * T.T_dp + T.T_opt + P.step_overhead;
    // what the pipeline time is priced with: tokens/s/GPU = tokens / ((T_pipe + rest) * world * taxes)
    float denom = (float)S.D.world;
    if (!P.kern[c.kv].is_native) denom *= 1.f + P.kern[c.kv].patch_ovh;
    if (S.D.ov) denom *= 1.f + sc.sched_ovh;
    if (S.D.ov && c.sh == PF_SHARD_ZERO1_OFFLOAD) denom *= 1.f + P.offload_overlap_penalty;
    r.denom = denom;
    r.hash = mix32(mix32(mix32(A.seed + 0x9e3779b9u) ^ (uint32_t)idx) ^ (uint32_t)(idx >> 32));
    r.w = (uint32_t)w;
    r.meta = sim_meta(c.pp, S.D.v_eff, S.D.kind, m_sim, ring);
    r.m = (uint32_t)(S.D.m > (RI)0xFFFFFFFFu ? (RI)0xFFFFFFFFu : S.D.m);
    r.pad[0] = r.pad[1] = r.pad[2] = r.pad[3] = 0u;
    const uint4 *src = reinterpret_cast<const uint4 *>(&r);
    uint4 *dst = reinterpret_cast<uint4 *>(
        A.recs + PF_AT(P.chk, A.bin_off[bin] + base + __popc(peers & ((1u << lane) - 1u)), A.n, PF_SITE_RECORD));
#pragma unroll
    for (int i = 0; i < 4; i++) dst[i] = src[i];
}

// The round loops, one per schedule class (all candidates of a batch share the class).  The timeline has one
// 32-bit word per (stage stream, microbatch), at index microbatch * streams + stream: 0 = nothing finished, +t =
// forward ended at t, -t = backward ended at t.  In every round a lane runs at most its next op, and only if the
// word it depends on already carries the right sign; a step's results are selected by that test, not branched
// around.  Every 64 rounds some lane of the warp must have
// advanced, otherwise the loop ends and the unfinished candidates are reported as stalled.
#define PF_SIM_ROUND_END()                                               \
    if (!__any_sync(0xFFFFFFFFu, done < total_ops)) break;               \
    if ((++rounds & 63) == 0) {                                          \
        if (!__any_sync(0xFFFFFFFFu, moved)) break;                      \
        moved = false;                                                   \
    }

// The static 1F1B and interleaved orders have one shape per rank: `warm` forward units, then forward / backward
// pairs, then the remaining backward units.  With nF forwards and nB backwards done, the next op is a forward
// iff nF < U and nF - nB <= warm, otherwise a backward.  One loop iteration therefore offers every lane a forward
// step and then a backward step, each straight-line code for its one kind of op; in the steady state a lane does
// both, so an iteration retires two ops for about the instructions one generic step would take.  A value written
// in a step is seen by the neighbour's next step of the same kind, one iteration later.
// (UL: the lane's unit count; once no lane of the warp has a forward left the loop is left for a backward-only one)
#define PF_SIM_ITER_END(UL)                                              \
    if (!__any_sync(0xFFFFFFFFu, nF < (UL))) break;                      \
    if ((++rounds & 63) == 0) {                                          \
        if (!__any_sync(0xFFFFFFFFu, nF + nB != seen)) break;            \
        seen = nF + nB;                                                  \
    }

// 1F1B: rank = stage = lane
// (chk, w_lim, r_lim: the checked build's record, the timeline's length for writes, the words from the timeline's
// start to the end of the warp's slice for reads)
__device__ __forceinline__ void sim_rounds_1f1b(volatile float *tl, const float *durF, const float *durB, int glane,
                                                int pp, int nj, int warm, int total_ops, float lat, int fonly,
                                                float &clock_out, int &done_out, unsigned int *chk, int w_lim,
                                                int r_lim, int sw)
{
    (void)chk; (void)w_lim; (void)r_lim;
    // lanes beyond the pipeline depth take no part: they poll row 0 and never act
    const bool active = total_ops > 0;
    const int row = active ? glane : 0;
    const bool depF = active && row > 0, depB = active && row < pp - 1;
    const float dF = active ? durF[row] : 0.f, dB = active ? durB[row] : 0.f;
    const float latF = depF ? lat : 0.f, latB = depB ? lat : 0.f;
    const int njl = active ? nj : 0;   // a lane beyond the pipeline depth has nothing to do
    int nF = 0, nB = 0, rounds = 0, seen = 0;
    float clock = 0.f;
    // microbatch-major timeline: word j * pp + stage.  aF / aB: the own word of the next forward / backward unit;
    // the word polled is its neighbour one stage down / up (the own word when there is no dependency)
    int aF = row, aB = row;
    const int pF = depF ? -1 : 0, pB = depB ? 1 : 0;
    // a step is straight-line code whose results are selected by its go / no-go predicate
    // (index nF may be nj once all forwards are done: that word lies inside the warp's slice)
#define PF_SIM_FWD(e)                                                                        \
    {                                                                                        \
        const bool go = nF < njl && nF - nB <= warm && (!depF || (e) > 0.f);                 \
        const float t = fmaxf(clock, depF ? (e) + latF : 0.f) + dF;                          \
        if (go) tl[PF_AT(chk, (aF) ^ sw, w_lim, PF_SITE_TIMELINE)] = t;                             \
        clock = go ? t : clock;                                                              \
        aF += go ? pp : 0;                                                                   \
        nF += go ? 1 : 0;                                                                    \
    }
#define PF_SIM_BWD(e)                                                                        \
    {                                                                                        \
        const bool go = nB < njl && (nF - nB > warm || nF == njl) && (!depB || (e) < 0.f);   \
        const float t = fmaxf(clock, depB ? latB - (e) : 0.f) + dB;                          \
        if (go) tl[PF_AT(chk, (aB) ^ sw, w_lim, PF_SITE_TIMELINE)] = -t;                            \
        clock = go ? t : clock;                                                              \
        aB += go ? pp : 0;                                                                   \
        nB += go ? 1 : 0;                                                                    \
    }
    // No backward can run before the first microbatch has crossed the shallowest pipeline of the warp: the first
    // `fonly` steps are forward steps only.
    for (int i = 0; i < fonly; i++) {
        const float eF = tl[PF_AT(chk, (aF + pF) ^ sw, r_lim, PF_SITE_TIMELINE)];
        PF_SIM_FWD(eF)
    }
    for (;;) {
#pragma unroll
        for (int rep = 0; rep < 2; rep++) {
            // both polls are issued before either step runs, so that their shared-memory latencies overlap (the
            // backward step's dependency is another lane's word: reading it a few instructions early only means a
            // value that arrives in between is seen one iteration later)
            const float eF = tl[PF_AT(chk, (aF + pF) ^ sw, r_lim, PF_SITE_TIMELINE)];
            const float eB = tl[PF_AT(chk, (aB + pB) ^ sw, r_lim, PF_SITE_TIMELINE)];
            PF_SIM_FWD(eF)
            PF_SIM_BWD(eB)
        }
        PF_SIM_ITER_END(njl)
    }
    // cool-down: every forward of the warp is done, only backward steps are left
    while (__any_sync(0xFFFFFFFFu, nB < njl)) {
#pragma unroll
        for (int rep = 0; rep < 4; rep++) {
            const float eB = tl[PF_AT(chk, (aB + pB) ^ sw, r_lim, PF_SITE_TIMELINE)];
            PF_SIM_BWD(eB)
        }
        if ((++rounds & 15) == 0) {
            if (!__any_sync(0xFFFFFFFFu, nF + nB != seen)) break;
            seen = nF + nB;
        }
    }
#undef PF_SIM_FWD
#undef PF_SIM_BWD
    clock_out = clock;
    done_out = nF + nB;
}

// Interleaved: v chunks per rank; unit k of a rank is microbatch (k / (pp v)) pp + k mod pp of chunk
// (k mod (pp v)) / pp, backward units walk the chunks downward.  Per direction a lane carries the timeline index of
// its next unit's own word and that unit's stage, and advances both by one of three precomputed steps (next
// microbatch of the window, next chunk, next window), chosen by two countdowns: no multiplications and no
// divisions in the loop, and a step is straight-line code whose results are selected by its go / no-go predicate.
__device__ __forceinline__ void sim_rounds_interleaved(volatile float *tl, const float *durF, const float *durB,
                                                       int glane, int pp, int v, int nj, int U, int warm,
                                                       int total_ops, float lat, int fonly, float &clock_out,
                                                       int &done_out, unsigned int *chk, int w_lim, int r_lim,
                                                       int q_lim, int sw)
{
    (void)chk; (void)w_lim; (void)r_lim; (void)q_lim;
    const int Q = pp * v;
    const bool active = total_ops > 0;
    const int row = active ? glane : 0;                    // lanes beyond the pipeline depth poll rank 0's rows
    const int Ul = active ? U : 0;                         // a lane beyond the pipeline depth has nothing to do
    int nF = 0, nB = 0, rounds = 0, seen = 0;
    float clock = 0.f;
    // forward cursor: chunk 0, window 0, microbatch 0; backward cursor: the last chunk first
    // microbatch-major timeline: word j * Q + stage (the lanes of a group touch neighbouring words: no bank conflicts)
    const int stepF_chunk = pp - (pp - 1) * Q, stepF_window = Q - (v - 1) * pp;   // next chunk: stage + pp, back to the window's first microbatch
    const int stepB_chunk = -pp - (pp - 1) * Q, stepB_window = Q + (v - 1) * pp;
    int aF = row, qF = row, fw = pp - 1, fc = v - 1;       // fw / fc: units left in the window / chunks left in the round
    int aB = (v - 1) * pp + row, qB = (v - 1) * pp + row, bw = pp - 1, bc = v - 1;
    // one forward step: the unit's dependency is the same microbatch one stage earlier (e: that word, read by the caller)
#define PF_SIM_FWD(e)                                                                                   \
    {                                                                                                   \
        const bool dep = qF > 0;                                                                        \
        const bool go = nF < Ul && nF - nB <= warm && (!dep || (e) > 0.f);                              \
        const float t = fmaxf(clock, dep ? (e) + lat : 0.f) + durF[PF_AT(chk, qF, q_lim, PF_SITE_DURATION)]; \
        if (go) tl[PF_AT(chk, (aF) ^ sw, w_lim, PF_SITE_TIMELINE)] = t;                                        \
        clock = go ? t : clock;                                                                         \
        const bool ww = fw == 0, wc = fc == 0;                                                          \
        aF += go ? (ww ? (wc ? stepF_window : stepF_chunk) : Q) : 0;                                    \
        qF += (go && ww) ? (wc ? -(v - 1) * pp : pp) : 0;                                               \
        fc = (go && ww) ? (wc ? v - 1 : fc - 1) : fc;                                                   \
        fw = go ? (ww ? pp - 1 : fw - 1) : fw;                                                          \
        nF += go ? 1 : 0;                                                                               \
    }
    // one backward step: the dependency is the same microbatch one stage later
#define PF_SIM_BWD(e)                                                                                   \
    {                                                                                                   \
        const bool dep = qB < Q - 1;                                                                    \
        const bool go = nB < Ul && (nF - nB > warm || nF == Ul) && (!dep || (e) < 0.f);                 \
        const float t = fmaxf(clock, dep ? lat - (e) : 0.f) + durB[PF_AT(chk, qB, q_lim, PF_SITE_DURATION)]; \
        if (go) tl[PF_AT(chk, (aB) ^ sw, w_lim, PF_SITE_TIMELINE)] = -t;                                       \
        clock = go ? t : clock;                                                                         \
        const bool ww = bw == 0, wc = bc == 0;                                                          \
        aB += go ? (ww ? (wc ? stepB_window : stepB_chunk) : Q) : 0;                                    \
        qB += (go && ww) ? (wc ? (v - 1) * pp : -pp) : 0;                                               \
        bc = (go && ww) ? (wc ? v - 1 : bc - 1) : bc;                                                   \
        bw = go ? (ww ? pp - 1 : bw - 1) : bw;                                                          \
        nB += go ? 1 : 0;                                                                               \
    }
    // the words polled: one stage down / up from the own word (the own word when there is no dependency; once a
    // direction has run out of units its cursor rests up to Q words past the timeline, inside the warp's slice)
#define PF_SIM_POLL_F() tl[PF_AT(chk, (aF - (qF > 0 ? 1 : 0)) ^ sw, r_lim, PF_SITE_TIMELINE)]
#define PF_SIM_POLL_B() tl[PF_AT(chk, (aB + (qB < Q - 1 ? 1 : 0)) ^ sw, r_lim, PF_SITE_TIMELINE)]
    // forward steps only until the first microbatch can have crossed the shallowest pipeline of the warp
    for (int i = 0; i < fonly; i++) {
        const float eF = PF_SIM_POLL_F();
        PF_SIM_FWD(eF)
    }
    for (;;) {
#pragma unroll
        for (int rep = 0; rep < 2; rep++) {
            // both polls first (see the 1F1B loop), then the two steps
            const float eF = PF_SIM_POLL_F();
            const float eB = PF_SIM_POLL_B();
            PF_SIM_FWD(eF)
            PF_SIM_BWD(eB)
        }
        PF_SIM_ITER_END(Ul)
    }
    // cool-down: every forward of the warp is done, only backward steps are left
    while (__any_sync(0xFFFFFFFFu, nB < Ul)) {
#pragma unroll
        for (int rep = 0; rep < 4; rep++) {
            const float eB = PF_SIM_POLL_B();
            PF_SIM_BWD(eB)
        }
        if ((++rounds & 15) == 0) {
            if (!__any_sync(0xFFFFFFFFu, nF + nB != seen)) break;
            seen = nF + nB;
        }
    }
#undef PF_SIM_FWD
#undef PF_SIM_BWD
#undef PF_SIM_POLL_F
#undef PF_SIM_POLL_B
    clock_out = clock;
    done_out = nF + nB;
}

// Interleaved on a ring timeline: W = 2 pp microbatch slots per stage stream, slot (j mod W) * Q + stage, two words
// per slot: a tag (2 j + 1 once the forward of microbatch j has ended, 2 j + 2 once its backward has) and the time.
// A reader takes a slot only when it carries exactly the tag it waits for, so a slot that was reused too early could
// only ever make a reader wait for ever -- which the no-progress check reports as a stall -- never hand it a wrong
// time.  The order's window of pp microbatches divides W, so a window never wraps inside: the ring row of unit
// (window g, position w) is (g & 1) pp + w, and the cursor steps are those of the full timeline except when an odd
// window is followed by an even one.
__device__ __forceinline__ void sim_rounds_interleaved_ring(volatile unsigned long long *tl, const float *durF,
                                                            const float *durB, int glane, int pp, int v, int U,
                                                            int warm, int total_ops, float lat, int fonly,
                                                            float &clock_out, int &done_out, unsigned int *chk,
                                                            int w_lim, int r_lim, int q_lim, int sw)
{
    (void)chk; (void)w_lim; (void)r_lim; (void)q_lim;
    const int Q = pp * v;
    const bool active = total_ops > 0;
    const int row = active ? glane : 0;
    const int Ul = active ? U : 0;
    int nF = 0, nB = 0, rounds = 0, seen = 0;
    float clock = 0.f;
    const int stepF_chunk = pp - (pp - 1) * Q, stepB_chunk = -pp - (pp - 1) * Q;
    // next window: one ring row up, or from the last row back to the first
    const int stepF_up = Q - (v - 1) * pp, stepF_wrap = -(2 * pp - 1) * Q - (v - 1) * pp;
    const int stepB_up = Q + (v - 1) * pp, stepB_wrap = -(2 * pp - 1) * Q + (v - 1) * pp;
    // slot of the next unit's own entry, its stage, its microbatch, countdowns, and whether its window is an odd one
    int aF = row, qF = row, jF = 0, fw = pp - 1, fc = v - 1, oddF = 0;
    int aB = (v - 1) * pp + row, qB = (v - 1) * pp + row, jB = 0, bw = pp - 1, bc = v - 1, oddB = 0;
#define PF_RING_WORD(tag, t) (((unsigned long long)__float_as_uint(t) << 32) | (unsigned int)(tag))
#define PF_SIM_FWD(e)                                                                                   \
    {                                                                                                   \
        const bool dep = qF > 0;                                                                        \
        const bool ready = !dep || (unsigned int)(e) == (unsigned int)(2 * jF + 1);                     \
        const bool go = nF < Ul && nF - nB <= warm && ready;                                            \
        const float ev = __uint_as_float((unsigned int)((e) >> 32));                                    \
        const float t = fmaxf(clock, dep ? ev + lat : 0.f) + durF[PF_AT(chk, qF, q_lim, PF_SITE_DURATION)]; \
        if (go) tl[PF_AT(chk, (aF) ^ sw, w_lim, PF_SITE_TIMELINE)] = PF_RING_WORD(2 * jF + 1, t);              \
        clock = go ? t : clock;                                                                         \
        const bool ww = fw == 0, wc = fc == 0;                                                          \
        aF += go ? (ww ? (wc ? (oddF ? stepF_wrap : stepF_up) : stepF_chunk) : Q) : 0;                  \
        jF += go ? (ww ? (wc ? 1 : -(pp - 1)) : 1) : 0;                                                 \
        oddF ^= (go && ww && wc) ? 1 : 0;                                                               \
        qF += (go && ww) ? (wc ? -(v - 1) * pp : pp) : 0;                                               \
        fc = (go && ww) ? (wc ? v - 1 : fc - 1) : fc;                                                   \
        fw = go ? (ww ? pp - 1 : fw - 1) : fw;                                                          \
        nF += go ? 1 : 0;                                                                               \
    }
#define PF_SIM_BWD(e)                                                                                   \
    {                                                                                                   \
        const bool dep = qB < Q - 1;                                                                    \
        const bool ready = !dep || (unsigned int)(e) == (unsigned int)(2 * jB + 2);                     \
        const bool go = nB < Ul && (nF - nB > warm || nF == Ul) && ready;                               \
        const float ev = __uint_as_float((unsigned int)((e) >> 32));                                    \
        const float t = fmaxf(clock, dep ? ev + lat : 0.f) + durB[PF_AT(chk, qB, q_lim, PF_SITE_DURATION)]; \
        if (go) tl[PF_AT(chk, (aB) ^ sw, w_lim, PF_SITE_TIMELINE)] = PF_RING_WORD(2 * jB + 2, t);              \
        clock = go ? t : clock;                                                                         \
        const bool ww = bw == 0, wc = bc == 0;                                                          \
        aB += go ? (ww ? (wc ? (oddB ? stepB_wrap : stepB_up) : stepB_chunk) : Q) : 0;                  \
        jB += go ? (ww ? (wc ? 1 : -(pp - 1)) : 1) : 0;                                                 \
        oddB ^= (go && ww && wc) ? 1 : 0;                                                               \
        qB += (go && ww) ? (wc ? (v - 1) * pp : -pp) : 0;                                               \
        bc = (go && ww) ? (wc ? v - 1 : bc - 1) : bc;                                                   \
        bw = go ? (ww ? pp - 1 : bw - 1) : bw;                                                          \
        nB += go ? 1 : 0;                                                                               \
    }
    // once a direction has run out of units its cursor rests on some slot of the ring: a valid word, never taken
#define PF_SIM_POLL_F() tl[PF_AT(chk, (aF - (qF > 0 ? 1 : 0)) ^ sw, r_lim, PF_SITE_TIMELINE)]
#define PF_SIM_POLL_B() tl[PF_AT(chk, (aB + (qB < Q - 1 ? 1 : 0)) ^ sw, r_lim, PF_SITE_TIMELINE)]
    for (int i = 0; i < fonly; i++) {
        const unsigned long long eF = PF_SIM_POLL_F();
        PF_SIM_FWD(eF)
    }
    for (;;) {
#pragma unroll
        for (int rep = 0; rep < 2; rep++) {
            const unsigned long long eF = PF_SIM_POLL_F();
            const unsigned long long eB = PF_SIM_POLL_B();
            PF_SIM_FWD(eF)
            PF_SIM_BWD(eB)
        }
        PF_SIM_ITER_END(Ul)
    }
    while (__any_sync(0xFFFFFFFFu, nB < Ul)) {
#pragma unroll
        for (int rep = 0; rep < 4; rep++) {
            const unsigned long long eB = PF_SIM_POLL_B();
            PF_SIM_BWD(eB)
        }
        if ((++rounds & 15) == 0) {
            if (!__any_sync(0xFFFFFFFFu, nF + nB != seen)) break;
            seen = nF + nB;
        }
    }
#undef PF_SIM_FWD
#undef PF_SIM_BWD
#undef PF_SIM_POLL_F
#undef PF_SIM_POLL_B
#undef PF_RING_WORD
    clock_out = clock;
    done_out = nF + nB;
}
#undef PF_SIM_ITER_END

// DualPipe-style: two directions; the per-rank order comes from the host-built table
__device__ __forceinline__ void sim_rounds_dual(volatile float *tl, const float *durF, const float *durB, int glane,
                                                int pp, int nj, const uint8_t *ops, int total_ops, float lat,
                                                float &clock_out, int &done_out, unsigned int *chk, int w_lim,
                                                int r_lim, int q_lim, int sw)
{
    (void)chk; (void)w_lim; (void)r_lim; (void)q_lim;
    int done = 0, rounds = 0;
    bool moved = false;
    float clock = 0.f;
    for (;;) {
#pragma unroll
        for (int rep = 0; rep < 4; rep++)
        if (done < total_ops) {
            const uint32_t op = __ldg(ops + PF_AT(chk, done, total_ops, PF_SITE_DUAL_OPS));
            const bool isb = op & 1;
            const int d = (op >> 1) & 1, j = op >> 2;
            const int q = d ? pp - 1 - glane : glane;
            const int sidx = d * pp + q;
            const bool dep = isb ? (q < pp - 1) : (q > 0);
            const int nb = dep ? (isb ? sidx + 1 : sidx - 1) : sidx;
            const float e = tl[PF_AT(chk, (j * 2 * pp + nb) ^ sw, r_lim, PF_SITE_TIMELINE)];
            const float dur = (isb ? durB : durF)[PF_AT(chk, q, q_lim, PF_SITE_DURATION)];
            if (!dep || (isb ? e < 0.f : e > 0.f)) {
                clock = fmaxf(clock, dep ? fabsf(e) + lat : 0.f) + dur;
                tl[PF_AT(chk, (j * 2 * pp + sidx) ^ sw, w_lim, PF_SITE_TIMELINE)] = isb ? -clock : clock;
                done++;
                moved = true;
            }
        }
        PF_SIM_ROUND_END()
    }
    clock_out = clock;
    done_out = done;
}
#undef PF_SIM_ROUND_END

// One launch serves every bin.  Every warp owns a fixed slice of the block's shared memory, large enough for
// one timeline of the largest class (or several of a smaller one), and draws batches from one queue that runs
// through the bins -- longest simulations first, so the tail is one candidate long.  No block-level barrier is
// involved after the queue's tables have been staged.
//
// Global memory is touched three times per batch and hardly on the critical path: the next batch's queue ticket
// is drawn while the current batch is simulated, its records are requested before the current results are reduced,
// and the results are stored without waiting.  That matters inside a search call, where this kernel shares the GPU with a
// saturated store stream under which every round trip to L2 takes microseconds.
//
// Inside a warp a candidate is run by a group of 4, 8, 16 or 32 lanes, lane = pipeline rank; a warp takes as many
// candidates per batch as it has groups and its slice has room.  Each lane walks its rank's fixed op order and
// computes  end(op) = max(rank clock, end(dependency) + latency) + duration.  A forward of stage q needs the
// forward of stage q-1 of the same microbatch, a backward of stage q the backward of stage q+1 (the op's own
// forward is already behind the lane's clock).  The timeline has ONE 32-bit word per (stage stream,
// microbatch): 0 while nothing has finished, +t once the forward has ended at t, -t once the backward has --
// the forward's end has been consumed by stage q+1 before the backward of the same slot can start, so the two
// never need the word at the same time.  The owner writes it, the neighbour polls it with a volatile load.  In
// every round a lane runs at most its next op; the body is branch-free apart from the readiness test, so lanes
// (and the groups of a warp) stay converged and a round costs one shared-memory poll plus one vote.  Every 64
// rounds some lane of the warp must have advanced, otherwise its unfinished candidates are reported as
// PF_SIM_STALL: the loop is bounded by the op count.
// Two instances: kRings = true serves the large calls (at least kSimRingMinSurvivors actual survivors: ring-timeline
// bins, four-lane groups, bank-permuted timelines); kRings = false is the same kernel without the ring loop and
// the permutation (fewer registers, fewer instructions per step), for all other calls.
template <bool kRings>
__global__ void __launch_bounds__(kSimThreads, 4) simulate_kernel(const __grid_constant__ DevPlan P, const SimArgs A)
{
    chain_enter();
    // which instance serves the call is decided here, from the actual number of survivors (the host knows only the
    // list's capacity and launches both when that is large)
    {
        uint64_t n_call = A.n;
        if (A.d_n) {
            const uint64_t dn = *A.d_n;
            n_call = dn < n_call ? dn : n_call;
        }
        if ((n_call >= kSimRingMinSurvivors) != kRings) return;
    }
    extern __shared__ __align__(16) float s_mem[];
    // (1,016 bytes, and not one more: three blocks of this kernel -- 72 KB of timelines each -- and one block of the fill
    // kernel fill an SM's shared memory to the last kilobyte)
    __shared__ unsigned int s_pre[kSimBins + 1], s_off[kSimBins + 1];
    __shared__ uint8_t s_seq[kSimBins];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int E_hi = sim_class_entries(A.cls_hi);
    for (int i = threadIdx.x; i <= kSimBins; i += kSimThreads) {
        if (i < kSimBins) s_seq[i] = (uint8_t)A.bin_seq[i];
        s_pre[i] = A.batch_pre[i];           // positions past the last bin hold no batches: entry kSimBins = all
        s_off[i] = A.bin_off[i];
    }
    __syncthreads();
    float *slice = s_mem + (size_t)warp * A.warp_floats;   // [E_hi] timelines, then the groups' (durF, durB) tables
    const unsigned int n_batches = s_pre[kSimBins];

    // a batch number -> its bin, its place in the bin, this lane's record
    struct Fetch {
        int bin;
        bool have;
        uint4 r[4];
    };
    auto locate = [&](unsigned int t, Fetch &f) {
        f.bin = -1;
        f.have = false;
        if (t >= n_batches) return;
        // position in the queue's bin order: how many positions end at or before t
        int pos = 0;
#pragma unroll
        for (int h = 0; h < kSimTab / 32; h++) {
            const int i = lane + 32 * h;
            pos += __popc(__ballot_sync(0xFFFFFFFFu, i < kSimBins && s_pre[i + 1] <= t));
        }
        f.bin = (int)s_seq[pos];
        const int gi = (f.bin / kSimKinds) % kSimGroups;
        const int g = sim_group_lanes(gi), batch = sim_bin_batch(f.bin, A.cls_hi);
        const unsigned int first = (t - s_pre[pos]) * (unsigned int)batch;
        const int gidx = lane / g;
        f.have = gidx < batch && first + gidx < s_off[f.bin + 1] - s_off[f.bin];
        if (f.have) {
            const uint4 *src = reinterpret_cast<const uint4 *>(
                A.recs + PF_AT(P.chk, s_off[f.bin] + first + gidx, s_off[kSimBins], PF_SITE_RECORD));
#pragma unroll
            for (int i = 0; i < 4; i++) f.r[i] = __ldcg(src + i);
        }
    };
    // lane 0 draws the tickets; a ticket is drawn when the batch before it starts, so that a warp commits to no
    // more than one batch ahead (the queue's last, short batches go to whoever is free)
    unsigned int tkt = 0;
    if (lane == 0) tkt = atomicAdd(A.work, 1u);
    Fetch cur, nxt;
    locate(__shfl_sync(0xFFFFFFFFu, tkt, 0), cur);

    while (cur.bin >= 0) {
        if (lane == 0) tkt = atomicAdd(A.work, 1u);   // the next ticket: in flight while this batch is simulated

        const int bin = cur.bin;
        const int cls = bin / (kSimGroups * kSimKinds), gi = (bin / kSimKinds) % kSimGroups;
        const int bin_kind = bin % kSimKinds;
        // (four-lane groups exist in the calls that have ring timelines only: the other instance is compiled for
        // groups of eight lanes and more, and reports a narrower bin -- there is none -- as stalled)
        const int g = kRings ? sim_group_lanes(gi) : max(sim_group_lanes(gi), 8);
        const int E = sim_class_entries(cls);
        const int batch = sim_bin_batch(bin, A.cls_hi);       // candidates this warp runs side by side
        const int gidx = lane / g, glane = lane - gidx * g;
        const bool group_on = gidx < batch;
        volatile float *tl = slice + (size_t)(group_on ? gidx : 0) * E;   // the timeline
        // The groups' timelines start a multiple of 32 words apart and, candidates of one bin being alike, the groups
        // tend to touch the same relative word at the same time: the same banks.  Every timeline index is therefore
        // XORed with a constant of the group (a permutation of the 32-word stretches of its own timeline) that moves
        // group i's lanes i * g * (words per lane) banks on: the groups of a warp then cover different banks.
        // (large calls only: a small call is bound by instruction issue along its longest op chain, and the XOR costs
        // it more than the conflicts do -- measured 0.151 against 0.139 ms)
        const int sw = kRings ? (gidx * g * (bin_kind == kSimKindRing ? 2 : 1)) & 31 : 0;
        const int qg = sim_group_stages(g, A.q_max);           // stages a group's duration tables hold
        float *durF = slice + E_hi + (size_t)(group_on ? gidx : 0) * 2 * qg, *durB = durF + qg;
        const bool have = cur.have;                            // this group's candidate exists

        // ---- the group's candidate, from its record
        const float F_l = __uint_as_float(cur.r[0].x), B_l = __uint_as_float(cur.r[0].y);
        const float F_ld = __uint_as_float(cur.r[0].z), B_ld = __uint_as_float(cur.r[0].w);
        const float headF = __uint_as_float(cur.r[1].x), lat_p = __uint_as_float(cur.r[1].y);
        const float rest = __uint_as_float(cur.r[1].z), denom = __uint_as_float(cur.r[1].w);
        const uint32_t cand_hash = cur.r[2].x, w = cur.r[2].y, meta = cur.r[2].z, m_all = cur.r[2].w;
        bool run = have;
        const int pp = run ? (int)(meta & 31u) + 1 : 1, v = run ? (int)((meta >> 5) & 7u) + 1 : 1;
        const int kind = run ? (int)((meta >> 8) & 3u) : PF_KIND_1F1B;
        const int m_sim = run ? (int)((meta >> 10) & 127u) : 1;
        const bool ring = run && ((meta >> 17) & 1u) != 0u;   // interleaved, on a ring timeline
        const bool dual = kind == PF_KIND_DUALPIPE;
        const int Q = dual ? pp : pp * v;
        const int nj = dual ? m_sim / 2 : m_sim;      // microbatches per stage stream
        const int n_entries = ring ? Q * sim_ring_slots(pp) * 2 : (dual ? 2 * Q : Q) * nj;   // timeline words
        // filed under a bin that cannot hold it: never happens for the pre-pass's records; reported, not overrun
        bool stalled = run && (n_entries > E || Q > qg || pp > g || (ring ? kSimKindRing : kind) != bin_kind ||
                              (!kRings && (ring || gi == 0)));
        if (stalled) run = false;

        // ---- stage durations (balanced layer split, head on the last stage, jitter), cleared timeline
        __syncwarp();
        if (run) {
            const int L_lo = P.L / Q, L_rem = P.L - L_lo * Q;
            for (int q = glane; q < Q; q += g) {
                const int nq_i = L_lo + (q < L_rem ? 1 : 0);
                const int start = q * L_lo + min(q, L_rem);              // first layer of the stage
                const int ndq = max(0, min(nq_i, P.L_dense - start));    // its leading dense layers
                const float nq = (float)(nq_i - ndq), nd = (float)ndq;
                const bool last = q == Q - 1;
                const int qd = (int)PF_AT(P.chk, q, qg, PF_SITE_DURATION);
                durF[qd] = (nq * F_l + nd * F_ld + (last ? headF : 0.f)) * jitter(cand_hash, q, 0);
                durB[qd] = (nq * B_l + nd * B_ld + (last ? P.bwd_factor * headF : 0.f)) * jitter(cand_hash, q, 1);
            }
            // clear the timeline with 16-byte stores (the slot is a multiple of four words, 16-byte aligned)
            {
                float4 *tl4 = reinterpret_cast<float4 *>(const_cast<float *>(tl));
                const int n4 = ((n_entries + 31) & ~31) >> 2;   // whole 32-word stretches: what the permuted indices reach
#pragma unroll 4
                for (int i = glane; i < n4; i += g) tl4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        __syncwarp();

        // ---- per-lane order state (1F1B is the one-chunk case of the unit cursors)
        const bool rank_active = run && glane < pp;
        const int U = dual ? 2 * nj : nj * v;          // forward units of this rank
        const int warm = kind == PF_KIND_INTERLEAVED ? min(2 * (pp - glane - 1) + (v - 1) * pp, U)
                                                     : min(pp - glane - 1, U);
        const uint8_t *dops = A.dual_ops;              // any valid address for lanes that do not use it
        if (dual && run) {
            const int off = __ldg(A.dual_off + pp * 33 + nj);
            if (off < 0) stalled = true, run = false;  // no table for this shape
            else dops = A.dual_ops + off + (size_t)glane * 2 * m_sim;
        }
        const int total_ops = (rank_active && run) ? 2 * U : 0;
        const float lat = run ? lat_p : 0.f;
        // limits for the checked build: writes stay inside the candidate's own timeline, reads inside the warp's slice
        // (a lane that has run out of ops still polls one word past its row)
        const int w_lim = run ? ((n_entries + 31) & ~31) : 1;
        const int r_lim = A.warp_floats - (group_on ? gidx : 0) * E;
        // a batch's candidates share the schedule class of their bin: one specialised loop per class
        int done = 0;
        float clock = 0.f;
        // forward-only steps at the start: one fewer than the stages of the shallowest pipeline in the warp
        int fonly = (run && !dual) ? Q - 1 : 0x7FFFFFFF;
        fonly = __reduce_min_sync(0xFFFFFFFFu, fonly);
        if (fonly == 0x7FFFFFFF) fonly = 0;
        if (kRings && bin_kind == kSimKindRing)
            // (two-word slots: the limits count slots)
            sim_rounds_interleaved_ring(reinterpret_cast<volatile unsigned long long *>(tl), durF, durB, glane, pp, v, U,
                                        warm, total_ops, lat, fonly, clock, done, P.chk, w_lim >> 1, r_lim >> 1, qg, sw >> 1);
        else if (bin_kind == PF_KIND_1F1B)
            sim_rounds_1f1b(tl, durF, durB, glane, pp, nj, warm, total_ops, lat, fonly, clock, done, P.chk, w_lim, r_lim, sw);
        else if (bin_kind == PF_KIND_INTERLEAVED)
            sim_rounds_interleaved(tl, durF, durB, glane, pp, v, nj, U, warm, total_ops, lat, fonly, clock, done, P.chk,
                                   w_lim, r_lim, qg, sw);
        else
            sim_rounds_dual(tl, durF, durB, glane, pp, nj, dops, total_ops, lat, clock, done, P.chk, w_lim, r_lim, qg, sw);
        if (done < total_ops) stalled = true;

        // the next batch's records are requested before this batch's results are reduced and stored
        locate(__shfl_sync(0xFFFFFFFFu, tkt, 0), nxt);

        // ---- makespan, steady-state extension beyond the window, pricing (reductions inside the group)
        float work = 0.f;
        if (rank_active && run) {
            if (dual) {
                work = 0.5f * (durF[glane] + durB[glane] + durF[pp - 1 - glane] + durB[pp - 1 - glane]);
            } else {
                for (int cc = 0; cc < v; cc++) work += durF[cc * pp + glane] + durB[cc * pp + glane];
            }
        }
        float span = rank_active ? clock : 0.f;
        int any_stall = stalled ? 1 : 0;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float s2 = __shfl_xor_sync(0xFFFFFFFFu, span, off);
            const float w2 = __shfl_xor_sync(0xFFFFFFFFu, work, off);
            const int a2 = __shfl_xor_sync(0xFFFFFFFFu, any_stall, off);
            if (off < g) {
                span = fmaxf(span, s2);
                work = fmaxf(work, w2);
                any_stall |= a2;
            }
        }
        if (glane == 0 && have) {
            int status = PF_SIM_OK;
            float tput_out = 0.f;
            if (any_stall) {
                status = PF_SIM_STALL;
            } else {
                float T_pipe = span;
                if (m_all > (uint32_t)m_sim) T_pipe += (float)(m_all - (uint32_t)m_sim) * work;
                tput_out = fdiv((float)(P.gbs * (i64)P.seq), (T_pipe + rest) * denom);
            }
            const uint32_t wo = (uint32_t)PF_AT(P.chk, w, A.n, PF_SITE_SIM_OUT);
            if (A.tput_sim) A.tput_sim[wo] = tput_out;
            if (A.status) A.status[wo] = (uint8_t)status;
        }
        __syncwarp();
        cur = nxt;
    }
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
    chain_enter();
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

DenseTopkLayout dense_topk_layout(int sm_count, uint64_t n, uint32_t k)
{
    DenseTopkLayout l;
    const uint64_t nn = n ? n : 1, kk = k ? k : 1;
    uint64_t tb = (n + kThreads - 1) / kThreads;
    uint64_t cap = (uint64_t)sm_count * 2;
    l.blocks = (int)(tb < 1 ? 1 : (tb > cap ? cap : tb));
    l.keys_max = (uint64_t)l.blocks * kk;
    if (l.keys_max > nn) l.keys_max = nn < kk ? kk : nn;
    l.tk = topk_layout(l.keys_max, k);
    return l;
}

int launch_dense_topk(const float *d_score, uint64_t n, const uint64_t *d_n, uint32_t k, const uint64_t *d_idx_map,
                      void *d_workspace, const DenseTopkLayout &lay, uint64_t *d_topk_idx, float *d_topk_score,
                      uint32_t *d_topk_count, cudaStream_t st, int *n_kernels, bool ctrl_cleared)
{
    uint8_t *tws = (uint8_t *)d_workspace;
    if (!ctrl_cleared) PF_CUDA_TRY(cudaMemsetAsync(tws + lay.tk.off_ctrl, 0, 256, st), "dense top-k: counter reset");
    DenseTopkArgs t;
    t.score = d_score; t.n = n; t.d_n = d_n; t.k = k;
    t.keys = (unsigned long long *)(tws + lay.tk.off_keys_a);
    t.key_count = (unsigned int *)(tws + lay.tk.off_ctrl) + 1;
    if (ctrl_cleared)
        launch_chained(dense_topk_kernel, lay.blocks, kThreads, 0, st, t);
    else
        dense_topk_kernel<<<lay.blocks, kThreads, 0, st>>>(t);
    count_launch();
    PF_CUDA_TRY(cudaGetLastError(), "dense_topk_kernel launch");
    int nk = 0;
    int rc = launch_topk_reduce(tws, lay.tk, lay.keys_max, k, 0, d_idx_map, d_topk_idx, d_topk_score, d_topk_count,
                                st, &nk, true);
    *n_kernels = nk + 1;
    return rc;
}

struct SimLayout {
    size_t off_ctrl, off_bin_of, off_recs, off_scores, off_topk, total;
    DenseTopkLayout dt;
};
constexpr size_t kSimCtrlBytes = 4096;   // work (64 words), bin_count, bin_off, bin_fill, bin_seq (kSimTab each), batch_pre
static_assert((64 + 5 * kSimTab + 1) * 4 <= 4096, "simulator control block");

static SimLayout sim_layout(const pf_plan_t *p, uint64_t n, uint32_t k)
{
    SimLayout l;
    const size_t nn = (size_t)(n ? n : 1);
    l.off_ctrl = 0;
    l.off_bin_of = kSimCtrlBytes;
    l.off_recs = l.off_bin_of + ((nn + 255) & ~(size_t)255);
    l.off_scores = l.off_recs + ((nn * sizeof(SimRec) + 255) & ~(size_t)255);
    l.off_topk = l.off_scores + ((nn * 4 + 255) & ~(size_t)255);
    l.dt = dense_topk_layout(p->sm_count, n, k);
    l.total = l.off_topk + (k ? l.dt.tk.total : 0);
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

// geometry of the simulator kernel for a plan: largest timeline class, a warp's slice, the pool of a block
struct SimGeom {
    int cls_hi, warp_floats, per_sm;
    size_t pool;
};
static SimGeom sim_geom(int q_max)
{
    SimGeom g;
    // largest class the plan can produce; a warp's slice holds one such timeline plus four duration tables
    const int entries_max = q_max * PF_SIM_WINDOW;
    g.cls_hi = 0;
    while (g.cls_hi < kSimClasses - 1 && sim_class_entries(g.cls_hi) < entries_max) g.cls_hi++;
    // a warp's slice: one timeline of the largest class, then the duration tables of as many lane groups as a warp holds
    int dur_floats = 0;
    for (int gi = 0; gi < kSimGroups; gi++) {
        const int lanes = sim_group_lanes(gi), need = (32 / lanes) * 2 * sim_group_stages(lanes, q_max);
        dur_floats = need > dur_floats ? need : dur_floats;
    }
    g.warp_floats = sim_class_entries(g.cls_hi) + ((dur_floats + 3) & ~3);
    g.pool = (size_t)(kSimThreads / 32) * g.warp_floats * sizeof(float);
    g.per_sm = (int)((size_t)(227 * 1024) / (g.pool + 1024 + 1280));
    g.per_sm = g.per_sm < 1 ? 1 : (g.per_sm > 12 ? 12 : g.per_sm);
    return g;
}

template <typename RI>
static int launch_simulate(pf_plan_t *p, SimArgs a, uint64_t n, cudaStream_t st, int *n_kernels)
{
    *n_kernels = 0;
    const SimGeom geo = sim_geom(a.q_max);
    if (geo.pool > 224 * 1024) return PF_EUNSUPPORTED;
    a.cls_hi = geo.cls_hi;
    a.warp_floats = geo.warp_floats;
    const unsigned int nb = (unsigned int)((n + 255) / 256);
    timing_begin(p, PF_T_SIMPREP, st);
    sim_classify_kernel<RI><<<nb, 256, 0, st>>>(p->dev, a);
    launch_chained(sim_offsets_kernel, 1, 32, 0, st, a);
    launch_chained(sim_records_kernel<RI>, nb, 256, 0, st, p->dev, a);
    for (int i = 0; i < 3; i++) count_launch();
    timing_end(p, PF_T_SIMPREP, 3, st);
    PF_CUDA_TRY(cudaGetLastError(), "simulator pre-pass launch");
    const uint64_t cap = (uint64_t)p->sm_count * geo.per_sm;
    const uint64_t want = (n + kSimThreads / 32 - 1) / (kSimThreads / 32);
    const int grid = (int)(want < cap ? want : cap);
    const int threads = kSimThreads;
    // Two instances (see simulate_kernel): a list that can hold kSimRingMinSurvivors gets both launches, and the one
    // that does not match the actual count ends at once.
    const bool both = n >= kSimRingMinSurvivors;
    PF_CUDA_TRY(ensure_dynamic_smem((const void *)simulate_kernel<false>, p->device, geo.pool), "simulate_kernel smem");
    if (both)
        PF_CUDA_TRY(ensure_dynamic_smem((const void *)simulate_kernel<true>, p->device, geo.pool), "simulate_kernel smem");
    timing_begin(p, PF_T_SIMULATE, st);
    if (both) {
        launch_chained(simulate_kernel<true>, grid, threads, geo.pool, st, p->dev, a);
        count_launch();
    }
    // (chained behind a running first instance, this one's blocks cannot land before blocks of that one leave: three
    // blocks of either fill an SM's shared memory)
    launch_chained(simulate_kernel<false>, grid, threads, geo.pool, st, p->dev, a);
    count_launch();
    timing_end(p, PF_T_SIMULATE, both ? 2 : 1, st);
    *n_kernels = both ? 5 : 4;
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
    return pf::simulate_run(p, d_surv_idx, n, d_n, jitter_seed, d_tput_sim, d_sim_status, k, d_topk_idx, d_topk_score,
                            d_topk_count, d_workspace, workspace_bytes, (cudaStream_t)stream);
}

int pf::simulate_run(pf_plan_t *p, const uint64_t *d_surv_idx, uint64_t n, const uint64_t *d_n, uint32_t jitter_seed,
                     float *d_tput_sim, uint8_t *d_sim_status, uint32_t k, uint64_t *d_topk_idx, float *d_topk_score,
                     uint32_t *d_topk_count, void *d_workspace, size_t workspace_bytes, cudaStream_t st)
{
    if (!p || !d_surv_idx) return PF_EINVAL;
    if (p->dev.phase != PF_PHASE_TRAIN) return PF_EUNSUPPORTED;
    if (k > PF_K_MAX) return PF_EINVAL;
    if (k > 0 && (!d_topk_idx || !d_topk_score || !d_topk_count)) return PF_EINVAL;
    if (n >= PF_MAX_COUNT) return PF_ERANGE;
    const SimLayout lay = sim_layout(p, n, k);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < lay.total) return PF_EWORKSPACE;
    if (!p->sim_tables) return PF_EINVAL;
    if (int rc_dev = check_device(p)) return rc_dev;
    int rc = PF_OK;
    const SimTables *tab = (const SimTables *)p->sim_tables;
    uint8_t *ws = (uint8_t *)d_workspace;
    float *scores = d_tput_sim ? d_tput_sim : (float *)(ws + lay.off_scores);

    SimArgs a;
    a.surv = d_surv_idx; a.n = n; a.d_n = d_n; a.seed = jitter_seed;
    a.tput_sim = scores; a.status = d_sim_status;
    a.work = (unsigned int *)(ws + lay.off_ctrl);
    a.bin_count = a.work + 64;
    a.bin_off = a.bin_count + kSimTab;
    a.bin_fill = a.bin_off + kSimTab;
    a.bin_seq = a.bin_fill + kSimTab;
    a.batch_pre = a.bin_seq + kSimTab;       // kSimTab + 1 words
    a.bin_of = ws + lay.off_bin_of;
    a.recs = (SimRec *)(ws + lay.off_recs);
    a.vals = p->d_vals; a.dual_ops = tab->d_ops; a.dual_off = tab->d_offset;
    a.q_max = plan_q_max(p);
    a.cls_hi = 0;
    a.warp_floats = 0;
    PF_CUDA_TRY(cudaMemsetAsync(ws + lay.off_ctrl, 0, kSimCtrlBytes, st), "pf_simulate: counter reset");
    // the re-ranking's counters too, here rather than in front of its kernel: nothing but kernels from here to the end,
    // each launch chained to the one before
    if (k > 0) PF_CUDA_TRY(cudaMemsetAsync(ws + lay.off_topk + lay.dt.tk.off_ctrl, 0, 256, st), "dense top-k: counter reset");
    if (n > 0) {
        int nk = 0;
        rc = p->dev.wide ? launch_simulate<unsigned long long>(p, a, n, st, &nk)
                         : launch_simulate<uint32_t>(p, a, n, st, &nk);
        if (rc != PF_OK) return rc;
    }
    // (inside a search call the fill stream is joined by the caller, after the re-ranking below, which does not read
    // the dense outputs)
    if (k > 0) {
        int nk = 0;
        timing_begin(p, PF_T_TOPK, st);
        rc = launch_dense_topk(scores, n, d_n, k, d_surv_idx, ws + lay.off_topk, lay.dt, d_topk_idx, d_topk_score,
                               d_topk_count, st, &nk, true);
        timing_end(p, PF_T_TOPK, nk, st);
        return rc;
    }
    return PF_OK;
}
