// pf_score.cu -- the scoring kernel (decode -> rules -> memory -> cost -> price -> block top-k), the top-k
// merge kernels, and their C entry points.
//
// Work decomposition.  The index space is cut into slabs: one slab = all combinations of the `n_inner`
// fastest-varying axes (<= 16384 candidates) for one combination of the remaining (outer) axes.  A
// persistent grid (four blocks per SM) draws tickets from an atomic counter; a table built by two small
// launches (and kept in the plan per range) maps tickets to slabs so that the slabs that must be evaluated
// come first, interleaved with a few constant ones, and the rest of the constant ones come last.
//   - Constant slab: a rule that depends on the outer axes alone fails, every candidate has the same reason;
//     the block streams that byte and zeros into the dense outputs with 16-byte stores.
//   - Evaluated slab: rules 4-7 go into a per-slab table over (sched, mb, v); inside a passing entry only the
//     kernel variant and the recompute mode vary, so rules 8-10 and the memory model are worked out once per
//     entry and looked up per candidate; the few candidates that pass the memory gate are queued and costed
//     one per thread.  The slab's outputs are written like a constant slab's: zeros up front, a reason image
//     collected in shared memory and copied out once, scattered patches only for gate-reaching candidates.
// Feasible candidates are offered to a shared-memory top-k buffer; each block appends its best keys to a
// compact list and the reduce kernels below finish the top-k.
#include "pf_eval.cuh"

namespace pf {

struct ScoreArgs {
    uint64_t first, count;          // range of this call
    uint64_t slab_lo;               // number of the first slab that intersects the range
    uint32_t n_slabs;               // slabs intersecting the range
    uint32_t slab_mul;              // visiting order: slab (s * slab_mul) mod n_slabs, slab_mul coprime to n_slabs
    uint32_t k;
    uint8_t *reason;
    float *tput;
    long long *mem;
    unsigned long long *keys;       // compact list of the blocks' best keys
    unsigned int *key_count;        // its length (zeroed before launch)
    unsigned long long *g_thr;      // largest k-th key any block has reached (zeroed before launch)
    unsigned int *slab_counter;     // zeroed before launch
    const int32_t *vals;            // packed axis value lists
    const int32_t *scen;            // serve: P[n_scen], O[n_scen]
    const uint32_t *order;          // ticket -> (pre_reason << 24) | slab, or NULL: visit by slab_mul, classify here
    const uint32_t *order_hdr;      // what the order table holds: slab_lo (2 words), n_slabs, tail, head length,
                                    // fills per evaluated slab
    uint32_t order_tail;            // the tail length this call wants
    uint32_t order_fpe;             // the fills per evaluated slab this call wants
    uint32_t head_only;             // 1: visit the head of the order only (tickets below hdr[4]); a second kernel
                                    // streams the constant slabs behind it
    ScoreDigest dg;                 // hist1 == NULL: not collected
};

// Per passing (sched, mb, v) entry of a slab: what its candidates share across kernel variant and recompute mode.
constexpr int kEntryBatch = kThreads / 4;
struct EntryInfo {
    long long mem[3];               // peak bytes per recompute mode
    uint32_t kv_bad;                // bit q: kernel variant q has no kernel for this entry's expert shape
    uint8_t unmapped;               // the schedule has no emitter mapping (and realizability is enforced)
    uint8_t rec_bad;                // bit r: recompute mode r breaks the overlap preconditions
};

struct SlabInfo {
    uint32_t slab;                  // slab number relative to slab_lo, or 0xFFFFFFFF when the queue is empty
    int pre_reason;                 // != 0: every candidate of the slab fails this rule
    int outer[PF_MAX_AXES];         // values of the outer axes (entries [n_inner, n_axes))
};

// Values of a slab's outer axes and, on request, the first failing rule among those that depend on the outer
// axes alone (0: the slab has to be evaluated candidate by candidate).
template <typename RI>
__device__ __forceinline__ int slab_outer_axes(const DevPlan &P, const int32_t *vals, uint64_t slab_abs,
                                               int (&outer)[PF_MAX_AXES], bool classify)
{
    uint64_t o = slab_abs;
    for (int a = P.n_inner; a < P.n_axes; a++) {
        uint64_t r = P.radix[a];
        uint64_t q = o / r;
        outer[a] = __ldg(vals + P.val_off[a] + (int)(o - q * r));
        o = q;
    }
    if (!classify || P.n_pre_rules <= 0) return 0;
    if (P.phase == PF_PHASE_TRAIN) {
        TrainTuple c;
        c.mb = P.n_inner <= 3 ? outer[3] : 1;
        c.ep = P.n_inner <= 5 ? outer[5] : 1;
        c.pp = outer[6]; c.tp = outer[7]; c.dp = outer[8]; c.world = outer[9];
        RI dp, world;
        int r = train_layout_rules<RI>(P, c, 1, P.n_pre_rules < 3 ? P.n_pre_rules : 3, dp, world);
        if (r == 0 && P.n_pre_rules >= 4) {
            RI dpmb = dp * (RI)c.mb;
            if (((RI)P.gbs) % dpmb != 0) r = PF_R_BATCH;
        }
        return r;
    }
    ServeTuple c;
    c.batch = P.n_inner <= 2 ? outer[2] : 1;
    c.dpa = outer[3]; c.ep = outer[4]; c.tp = outer[5];
    return serve_layout_rules<RI>(P, c, 1, P.n_pre_rules >= 4);
}

// Visiting order of a call's slabs.  A slab that has to be evaluated takes several times as long as one that is
// filled with a constant, so the evaluated ones go first, spread evenly between the filled ones (their
// arithmetic then runs under the other blocks' store traffic), and the last tickets are all fills: the kernel's
// tail is one short slab long.
//
// Step 1, one thread per slab: the slab's class (its pre_reason byte).
template <typename RI>
__global__ void __launch_bounds__(256) slab_class_kernel(const __grid_constant__ DevPlan P, const int32_t *vals,
                                                         uint64_t slab_lo, uint32_t n_slabs, uint8_t *cls)
{
    const uint32_t s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n_slabs) return;
    int outer[PF_MAX_AXES];
    cls[s] = (uint8_t)slab_outer_axes<RI>(P, vals, slab_lo + s, outer, true);
}

// Step 2, one block: ranks within each class by a block-wide scan over per-thread chunks, then every slab's
// ticket in closed form.  With H evaluated and F filled slabs, Fs = min(kFillsPerEvaluated * H, F - tail) fills
// are interleaved with the evaluated slabs (measured best: three or four fills per evaluated slab, i.e. about
// half of the blocks evaluating while the rest keep the store stream going) and the other fills follow: evaluated slab i sits after floor(i * Fs / H)
// fills, fill j < Fs after min(H, ceil((j + 1) * H / Fs)) evaluated slabs.
__global__ void __launch_bounds__(1024) slab_order_kernel(const uint8_t *cls, uint64_t slab_lo, uint32_t n_slabs,
                                                          uint32_t tail, uint32_t fpe, uint32_t *order, uint32_t *hdr)
{
    __shared__ uint32_t s_part[1024];
    const uint32_t tid = threadIdx.x;
    const uint32_t chunk = (n_slabs + 1023u) / 1024u;
    const uint32_t lo = min(tid * chunk, n_slabs), hi = min(lo + chunk, n_slabs);
    uint32_t h = 0;
    for (uint32_t s = lo; s < hi; s++) h += cls[s] == 0;
    s_part[tid] = h;
    __syncthreads();
    for (uint32_t d = 1; d < 1024u; d <<= 1) {  // inclusive scan
        const uint32_t v = tid >= d ? s_part[tid - d] : 0u;
        __syncthreads();
        s_part[tid] += v;
        __syncthreads();
    }
    const uint64_t H = s_part[1023], F = n_slabs - H;
    uint64_t Fs = F > tail ? F - tail : 0;
    if (Fs > H * fpe) Fs = H * fpe;
    uint64_t hi_rank = s_part[tid] - h;        // evaluated slabs before this chunk
    uint64_t fi_rank = lo - hi_rank;           // filled slabs before this chunk
    for (uint32_t s = lo; s < hi; s++) {
        const uint32_t c = cls[s];
        uint64_t pos;
        if (c == 0) {
            pos = hi_rank + (H ? hi_rank * Fs / H : 0);
            hi_rank++;
        } else {
            if (fi_rank < Fs) {
                uint64_t before = ((fi_rank + 1) * H + Fs - 1) / Fs;
                pos = fi_rank + (before < H ? before : H);
            } else {
                pos = H + fi_rank;
            }
            fi_rank++;
        }
        order[pos] = (c << 24) | s;
    }
    // the header names the range this table now holds; a reader that wants another range ignores the table
    if (tid == 0) {
        hdr[0] = (uint32_t)slab_lo;
        hdr[1] = (uint32_t)(slab_lo >> 32);
        hdr[2] = n_slabs;
        hdr[3] = tail;
        hdr[4] = (uint32_t)(H + Fs);   // the head: every evaluated slab and the fills interleaved with them
        hdr[5] = fpe;
    }
}

// Fill n bytes at p with byte b using 16-byte streaming stores where alignment allows.  Block-collective.
__device__ __forceinline__ void block_fill(uint8_t *p, uint64_t n, uint32_t b)
{
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    uint64_t head = (16 - ((uintptr_t)p & 15)) & 15;
    if (head > n) head = n;
    for (uint64_t i = tid; i < head; i += nt) p[i] = (uint8_t)b;
    const uint32_t w = b * 0x01010101u;
    const uint4 v = make_uint4(w, w, w, w);
    uint4 *q = reinterpret_cast<uint4 *>(p + head);
    const uint64_t nv = (n - head) >> 4;
    for (uint64_t i = tid; i < nv; i += nt) __stcs(q + i, v);
    const uint64_t done = head + (nv << 4);
    for (uint64_t i = done + tid; i < n; i += nt) p[i] = (uint8_t)b;
}

// Copy n bytes from shared memory to global memory, src and dst at the same offset modulo 16, with 16-byte
// streaming stores for the aligned body.  Block-collective.
__device__ __forceinline__ void block_copy_out(uint8_t *dst, const uint8_t *src, uint32_t n)
{
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    uint32_t head = (16u - (uint32_t)(reinterpret_cast<uintptr_t>(dst) & 15u)) & 15u;
    if (head > n) head = n;
    for (uint32_t i = tid; i < head; i += nt) dst[i] = src[i];
    const uint32_t nv = (n - head) >> 4;
    const uint4 *s4 = reinterpret_cast<const uint4 *>(src + head);
    uint4 *d4 = reinterpret_cast<uint4 *>(dst + head);
    for (uint32_t i = tid; i < nv; i += nt) __stcs(d4 + i, s4[i]);
    for (uint32_t i = head + (nv << 4) + tid; i < n; i += nt) dst[i] = src[i];
}

// One queued candidate through the memory model, the gate, the step-time model and the price.
struct CostOut {
    long long mem;
    float tput;
    int reason, v_eff;
};
template <typename RI>
__device__ __noinline__ CostOut train_cost(const DevPlan &P, const TrainTuple c)
{
    CostOut o;
    o.reason = 0;
    o.tput = 0.f;
    RI dp, world;
    TrainDerived<RI> D;
    train_layout_rules<RI>(P, c, 4, 3, dp, world);      // derives dp / world only
    train_plan_rules<RI>(P, c, dp, world, 4, D);        // the rules passed in phase 1: fills D
    TrainMem M;
    train_memory<RI>(P, c, D, M);
    o.mem = M.mem;
    o.v_eff = D.v_eff;
    if (M.mem > P.budget_bytes) {
        o.reason = PF_R_MEMORY;
    } else {
        TrainTimes T;
        train_times<RI>(P, c, D, M, T);
        o.tput = train_price<RI>(P, c, D, T, train_pipe_analytic<RI>(P, c, D, T));
        if (domain_why<RI>(P, P.kern[c.kv], D.m_e)) o.reason = PF_FLAG_EXTRAPOLATED;
    }
    return o;
}

template <typename RI>
__global__ void __launch_bounds__(kThreads, 4) score_kernel(const __grid_constant__ DevPlan P, const ScoreArgs A)
{
    chain_enter();
    __shared__ unsigned long long s_buf[kTopkCap];
    __shared__ int s_count;
    __shared__ unsigned long long s_thr;
    __shared__ SlabInfo s_slabs[2];
    __shared__ int s_base[2];
    __shared__ unsigned long long s_gthr;   // snapshot of the grid-wide threshold, refreshed once per slab
    __shared__ uint8_t s_tab[2048];         // rules 4-7 per (sched, mb, v) combination of the current slab
    __shared__ int32_t s_vals[kInnerVals];  // value lists of the inner axes (the packed array's prefix)
    __shared__ uint16_t s_pass[2048];       // table entries of the current slab that pass rules 4-7
    __shared__ int s_np;
    __shared__ EntryInfo s_info[kEntryBatch];  // what a batch of passing entries shares across kv and rec
    __shared__ int s_qn;                    // candidates of the current slab queued for the cost model
    // training plans: reason bytes of the current slab (P.slab + 16 bytes), then the queue of positions in the
    // slab that go to the cost model (kQueueCap entries, drained whenever it may fill up)
    extern __shared__ __align__(16) uint8_t s_dyn[];
    uint8_t *const s_img = s_dyn;
    uint16_t *const s_queue = reinterpret_cast<uint16_t *>(s_dyn + ((P.slab + 16 + 15) & ~15u));

    const int tid = threadIdx.x;
    const bool train = P.phase == PF_PHASE_TRAIN;
    const bool want_topk = A.k > 0;
    if (tid == 0) {
        s_count = 0;
        s_thr = 0ull;
    }
    // iterations that may still append without overflowing the buffer (one key per thread per iteration)
    int room_iters = kTopkCap / kThreads;
    unsigned long long thr = 0ull;

    // The inner axes' value lists are read once per candidate: keep them in shared memory.  Under the
    // store stream of the fill slabs a read that misses L1 waits thousands of cycles in L2.
    const int n_inner_vals = P.n_inner < P.n_axes ? P.val_off[P.n_inner] : P.val_off[P.n_axes - 1] + (int)P.radix[P.n_axes - 1];
    const bool vals_in_smem = n_inner_vals <= kInnerVals;
    if (vals_in_smem)
        for (int i = tid; i < n_inner_vals; i += kThreads) s_vals[i] = A.vals[i];
    const int32_t *inner_vals = vals_in_smem ? s_vals : A.vals;
    // Slab tickets run two ahead.  Under the store stream an atomic or a load that goes to L2 takes microseconds,
    // so thread 0 never waits for one where it was issued: the ticket drawn at the top of one slab is first
    // used at the top of the next one (to load its order word), and that word is first used at the bottom of
    // the same slab, after thread 0's share of the slab's stores, to set up the following slab.
    // The order table belongs to the plan and holds one range: use it only if that is this call's range.
    const uint32_t *order = nullptr;
    if (A.order && order_table_valid(A.order_hdr, A.slab_lo, A.n_slabs, A.order_tail, A.order_fpe)) order = A.order;
    // tickets this launch serves: the whole order, or its head when a fill kernel follows (without a valid table
    // this launch does everything and the fill kernel, which makes the same test, nothing)
    const uint32_t n_tickets = (order && A.head_only) ? A.order_hdr[4] : A.n_slabs;
    auto resolve = [&](uint32_t s, uint32_t w, SlabInfo &dst) {
        SlabInfo si;
        si.slab = 0xFFFFFFFFu;
        si.pre_reason = 0;
        if (s < n_tickets) {
            if (order) {
                // the visiting order and every slab's class were prepared by the launches before this one
                si.slab = w & 0xFFFFFFu;
                si.pre_reason = (int)(w >> 24);
                if (si.pre_reason == 0) slab_outer_axes<RI>(P, A.vals, A.slab_lo + si.slab, si.outer, false);
            } else {
                // too many slabs for an order table: a multiplicative permutation interleaves evaluated and
                // filled slabs, which cluster in index order
                si.slab = (uint32_t)(((uint64_t)s * A.slab_mul) % A.n_slabs);
                si.pre_reason = slab_outer_axes<RI>(P, A.vals, A.slab_lo + si.slab, si.outer, true);
            }
        }
        dst = si;
    };
    uint32_t tkt_next = 0, tkt_after = 0, word_next = 0;  // thread 0: tickets and order word in flight
    unsigned long long gthr_next = 0ull;                   // thread 0: the grid-wide threshold, in flight
    if (tid == 0) {
        // the first gridDim.x tickets are handed out by block number, the counter serves the ones after them
        const uint32_t t0 = blockIdx.x;
        s_gthr = 0ull;
        tkt_next = gridDim.x + atomicAdd(A.slab_counter, 1u);
        resolve(t0, (order && t0 < n_tickets) ? __ldcg(order + PF_AT(P.chk, t0, A.n_slabs, PF_SITE_ORDER)) : 0u, s_slabs[0]);
    }
    __syncthreads();

    for (int cur = 0;; cur ^= 1) {
        const SlabInfo &s_slab = s_slabs[cur];
        if (s_slab.slab == 0xFFFFFFFFu) break;
        if (tid == 0) {
            word_next = (order && tkt_next < n_tickets) ? __ldcg(order + PF_AT(P.chk, tkt_next, A.n_slabs, PF_SITE_ORDER)) : 0u;
            tkt_after = gridDim.x + atomicAdd(A.slab_counter, 1u);
            // the grid-wide threshold only matters to evaluated slabs: refresh it on those
            if (want_topk && s_slab.pre_reason == 0) gthr_next = *reinterpret_cast<volatile unsigned long long *>(A.g_thr);
        }
        // end of a slab: set up the next one from what was requested at its top
        auto finish_slab = [&]() {
            if (tid == 0) {
                resolve(tkt_next, word_next, s_slabs[cur ^ 1]);
                tkt_next = tkt_after;
                s_gthr = gthr_next;
            }
            __syncthreads();  // the next slab's record is complete and this one's no longer read
        };

        // candidate range of this slab clipped to the call's range
        const uint64_t slab_no = A.slab_lo + s_slab.slab;
        const uint64_t base = slab_no * (uint64_t)P.slab;
        const uint64_t lo = base > A.first ? base : A.first;
        const uint64_t end_slab = base + P.slab, end_call = A.first + A.count;
        const uint64_t hi = end_slab < end_call ? end_slab : end_call;
        const uint64_t rel0 = lo - A.first;  // offset of the first candidate in the dense outputs
        const uint32_t n = (uint32_t)(hi - lo);
        (void)PF_AT(P.chk, rel0 + n - 1, A.count, PF_SITE_DENSE);   // the slab's whole span lies inside the outputs

        if (s_slab.pre_reason != 0) {
            if (A.reason) block_fill(A.reason + rel0, n, (uint32_t)s_slab.pre_reason);
            if (A.tput) block_fill(reinterpret_cast<uint8_t *>(A.tput + rel0), (uint64_t)n * 4, 0u);
            if (A.mem) block_fill(reinterpret_cast<uint8_t *>(A.mem + rel0), (uint64_t)n * 8, 0u);
            finish_slab();
            continue;
        }

        const uint32_t j0 = (uint32_t)(lo - base);
        const int first_rule = P.n_pre_rules + 1;
        const bool use_tab = train && P.tab_n[0] > 0;
        if (use_tab) {
            const int n2 = P.tab_n[0], n3 = P.tab_n[1], n4 = P.tab_n[2];
            for (int e = tid; e < n2 * n3 * n4; e += kThreads) {
                const int d2 = e % n2, d3 = (e / n2) % n3, d4 = e / (n2 * n3);
                TrainTuple c;
                c.kv = 0; c.rec = 0;
                c.s = P.n_inner > 2 ? inner_vals[P.val_off[2] + d2] : s_slab.outer[2];
                c.mb = P.n_inner > 3 ? inner_vals[P.val_off[3] + d3] : s_slab.outer[3];
                c.v = P.n_inner > 4 ? inner_vals[P.val_off[4] + d4] : s_slab.outer[4];
                c.ep = s_slab.outer[5]; c.pp = s_slab.outer[6]; c.tp = s_slab.outer[7];
                c.dp = s_slab.outer[8]; c.world = s_slab.outer[9];
                c.sh = P.n_axes > 10 ? s_slab.outer[10] : PF_SHARD_ZERO1;
                RI dp, world;
                int r = train_layout_rules<RI>(P, c, first_rule, 3, dp, world);
                if (r == 0) {
                    TrainDerived<RI> D;
                    r = train_plan_rules<RI>(P, c, dp, world, first_rule, D, 7);
                }
                s_tab[PF_AT(P.chk, e, 2048, PF_SITE_TABLE)] = (uint8_t)r;
            }
            __syncthreads();
        }
        // inner digits by multiply-high division (exact: j * radix < 2^32)
        auto decode_inner = [&](uint32_t j, int (&v)[PF_MAX_AXES], int (&dg)[5]) {
            uint32_t rem = j;
#pragma unroll
            for (int a = 0; a < PF_MAX_AXES; a++) {
                if (a < P.n_inner) {
                    uint32_t r = P.radix[a];
                    uint32_t q = r == 1u ? rem : __umulhi(rem, P.magic[a]);
                    const int digit = (int)(rem - q * r);
                    if (a < 5) dg[a] = digit;
                    v[a] = inner_vals[PF_AT(P.chk, P.val_off[a] + digit, n_inner_vals, PF_SITE_VALS)];
                    rem = q;
                } else {
                    v[a] = a < P.n_axes ? s_slab.outer[a] : 0;
                }
            }
        };
        // offer a scored candidate to the block's top-k buffer (block-collective, once per iteration)
        auto offer = [&](bool feasible, float tput, uint32_t rel) {
            if (!want_topk) return;
            if (room_iters == 0) {
                __syncthreads();
                if (s_count > kTopkCap - kThreads) {
                    tk_prune<kTopkCap / 2 / kThreads>(s_buf, &s_count, &s_thr, (int)A.k);
                    // a block's k-th key bounds the global k-th from below: share it
                    if (tid == 0 && s_thr != 0ull) atomicMax(A.g_thr, s_thr);
                }
                room_iters = (kTopkCap - s_count) / kThreads;
                thr = s_thr > s_gthr ? s_thr : s_gthr;
                __syncthreads();
            }
            tk_push(s_buf, &s_count, thr, feasible, make_key(tput, rel));
            room_iters--;
        };

        if (train) {
            // Under the store stream of the fill slabs every store instruction of a warp waits a few hundred
            // nanoseconds whatever its width, so an evaluated slab writes as few and as wide stores as a filled
            // one: tput and mem are zeroed up front with 16-byte stores and only the candidates that reach the
            // cost model are patched; reason bytes are collected in a shared-memory image of the slab (laid
            // out at the same 16-byte phase as its destination) and copied out once at the end.
            const uint32_t pad = A.reason ? (uint32_t)(reinterpret_cast<uintptr_t>(A.reason + rel0) & 15u) : 0u;
            uint8_t *img = s_img + pad;
            if (A.tput) block_fill(reinterpret_cast<uint8_t *>(A.tput + rel0), (uint64_t)n * 4, 0u);
            if (A.mem) block_fill(reinterpret_cast<uint8_t *>(A.mem + rel0), (uint64_t)n * 8, 0u);
            if (tid == 0) {
                s_qn = 0;
                s_np = 0;
            }
            __syncthreads();
            // Phase 2 (block-collective): memory model, gate, step time and pricing for the queued candidates,
            // one per thread, every warp full; empties the queue.
            auto drain = [&]() {
                const uint32_t qn = (uint32_t)s_qn;
                for (uint32_t it = 0; it < qn; it += kThreads) {
                    const uint32_t qi = it + tid;
                    const bool active = qi < qn;
                    int reason = 0;
                    float tput = 0.f;
                    uint32_t i = 0;
                    if (active) {
                        i = s_queue[PF_AT(P.chk, qi, kQueueCap, PF_SITE_QUEUE)];
                        int v[PF_MAX_AXES], dg[5] = {0, 0, 0, 0, 0};
                        decode_inner(j0 + i, v, dg);
                        TrainTuple c;
                        c.kv = v[0]; c.rec = v[1]; c.s = v[2]; c.mb = v[3]; c.v = v[4];
                        c.ep = v[5]; c.pp = v[6]; c.tp = v[7]; c.dp = v[8]; c.world = v[9];
                        c.sh = P.n_axes > 10 ? v[10] : PF_SHARD_ZERO1;
                        // memory model, gate, step time and price in a function of its own (its registers are
                        // then allocated apart from this kernel's many live values)
                        const CostOut co = train_cost<RI>(P, c);
                        reason = co.reason;
                        tput = co.tput;
                        struct { long long mem; } M = {co.mem};
                        struct { int v_eff; } D = {co.v_eff};
                        const uint64_t o = PF_AT(P.chk, rel0 + i, A.count, PF_SITE_DENSE);
                        img[PF_AT(P.chk, pad + i, P.slab + 16, PF_SITE_IMAGE) - pad] = (uint8_t)reason;
                        if (A.tput && tput != 0.f) A.tput[o] = tput;
                        if (A.mem) A.mem[o] = M.mem;
                        // the selection's first pass, done here for the few feasible plans inside the simulator's
                        // domain: score-bit histograms, the chunk's eligible count, the list of non-empty chunks
                        if (A.dg.hist1 && tput != 0.f && c.pp <= PF_SIM_MAX_RANKS && D.v_eff <= PF_SIM_MAX_V) {
                            // lanes of the warp that add to the same word do it in one atomic (a slab's plans share
                            // a chunk or two and most of their score's leading bits): where many plans are feasible
                            // these atomics, issued under a saturated store stream, are what the drain waits for
                            const uint32_t bits = __float_as_uint(tput);
                            const int lane2 = tid & 31;
                            const unsigned here = __activemask();
                            const uint32_t n_chunks = (uint32_t)((A.count + A.dg.chunk - 1) / A.dg.chunk);
                            (void)n_chunks;
                            const uint32_t chunk = (uint32_t)PF_AT(P.chk, o / A.dg.chunk, n_chunks, PF_SITE_CHUNK);
                            const unsigned p1 = __match_any_sync(here, bits >> 16);
                            if (lane2 == __ffs(p1) - 1)
                                atomicAdd(A.dg.hist1 + PF_AT(P.chk, bits >> 16, 65536, PF_SITE_DIGEST), (unsigned)__popc(p1));
                            const unsigned p2 = __match_any_sync(here, bits >> 24);
                            if (lane2 == __ffs(p2) - 1)
                                atomicAdd(A.dg.coarse1 + PF_AT(P.chk, bits >> 24, 256, PF_SITE_DIGEST), (unsigned)__popc(p2));
                            const unsigned p3 = __match_any_sync(here, chunk);
                            if (lane2 == __ffs(p3) - 1 && atomicAdd(A.dg.elig + chunk, (unsigned)__popc(p3)) == 0u)
                                A.dg.list[PF_AT(P.chk, atomicAdd(A.dg.n_list, 1u), n_chunks, PF_SITE_CHUNK)] = chunk;
                        }
                    }
                    offer(active && (reason & 0x7f) == 0, tput, (uint32_t)(rel0 + i));
                }
                __syncthreads();
                if (tid == 0) s_qn = 0;
                __syncthreads();
            };
            // append this thread's candidate (position i in the clipped slab) to the queue; warp-collective
            auto enqueue = [&](bool queued, uint32_t i) {
                const unsigned mask = __ballot_sync(0xFFFFFFFFu, queued);
                if (mask) {
                    const int lane2 = tid & 31, leader = __ffs(mask) - 1;
                    int qb = 0;
                    if (lane2 == leader) qb = atomicAdd(&s_qn, __popc(mask));
                    qb = __shfl_sync(0xFFFFFFFFu, qb, leader);
                    if (queued)
                        s_queue[PF_AT(P.chk, qb + __popc(mask & ((1u << lane2) - 1u)), kQueueCap, PF_SITE_QUEUE)] = (uint16_t)i;
                }
            };
            int since_drain = 0;  // iterations that appended (at most kThreads entries each) since the last drain
            if (use_tab) {
                // Phase 1a.  Candidates that share (sched, mb, v) are contiguous: a run of R = |kv| x |rec|
                // indices.  A warp takes 32 table entries at a time; runs whose entry holds a failing rule get
                // their reason bytes at once; passing entries are only listed.
                const uint32_t n_combos = (uint32_t)(P.tab_n[0] * P.tab_n[1] * P.tab_n[2]);
                const uint32_t R = P.slab / n_combos;
                const int lane = tid & 31;
                for (uint32_t cb = 0; cb < n_combos; cb += kThreads) {
                    const uint32_t e = cb + tid;
                    const int t = e < n_combos ? (int)s_tab[PF_AT(P.chk, e, 2048, PF_SITE_TABLE)] : 0xFF;
                    const unsigned pm = __ballot_sync(0xFFFFFFFFu, t == 0);
                    if (pm) {
                        const int leader = __ffs(pm) - 1;
                        int pb = 0;
                        if (lane == leader) pb = atomicAdd(&s_np, __popc(pm));
                        pb = __shfl_sync(0xFFFFFFFFu, pb, leader);
                        if (t == 0) s_pass[PF_AT(P.chk, pb + __popc(pm & ((1u << lane) - 1u)), 2048, PF_SITE_PASS)] = (uint16_t)e;
                    }
                    if (t != 0 && t != 0xFF) {
                        // the run's candidates, clipped to the call's range
                        const uint32_t ja = max(e * R, j0), jb = min(e * R + R, j0 + n);
                        for (uint32_t j = ja; j < jb; j++)
                            img[PF_AT(P.chk, pad + j - j0, P.slab + 16, PF_SITE_IMAGE) - pad] = (uint8_t)t;
                    }
                }
                __syncthreads();
                // Phase 1b.  Inside a passing entry only the kernel variant and the recompute mode vary.  One
                // thread per entry works out what depends on neither: which variants lack a kernel at this
                // expert shape (rule 8), whether the schedule is unmapped (9), which recompute modes break the
                // overlap preconditions (10), and the peak memory per recompute mode (the variant does not
                // enter it).  The entry's candidates then only look these up; the few that pass the memory
                // gate are queued for the cost model.
                const uint32_t np = (uint32_t)s_np;
                for (uint32_t b0 = 0; b0 < np; b0 += kEntryBatch) {
                    const uint32_t nb = min((uint32_t)kEntryBatch, np - b0);
                    if ((uint32_t)(tid >> 2) < nb) {
                        // four lanes per entry: lanes 0-2 take one recompute mode's memory each, lane 3 the rules
                        const int role = tid & 3, slot = tid >> 2;
                        const int e = s_pass[PF_AT(P.chk, b0 + slot, 2048, PF_SITE_PASS)];
                        const int n2 = P.tab_n[0], n3 = P.tab_n[1];
                        const int d2 = e % n2, d3 = (e / n2) % n3, d4 = e / (n2 * n3);
                        TrainTuple c;
                        c.kv = 0; c.rec = role < 3 ? role : 0;
                        c.s = P.n_inner > 2 ? inner_vals[P.val_off[2] + d2] : s_slab.outer[2];
                        c.mb = P.n_inner > 3 ? inner_vals[P.val_off[3] + d3] : s_slab.outer[3];
                        c.v = P.n_inner > 4 ? inner_vals[P.val_off[4] + d4] : s_slab.outer[4];
                        c.ep = s_slab.outer[5]; c.pp = s_slab.outer[6]; c.tp = s_slab.outer[7];
                        c.dp = s_slab.outer[8]; c.world = s_slab.outer[9];
                        c.sh = P.n_axes > 10 ? s_slab.outer[10] : PF_SHARD_ZERO1;
                        RI dp, world;
                        TrainDerived<RI> D;
                        train_layout_rules<RI>(P, c, 4, 3, dp, world);   // derives dp / world only
                        train_plan_rules<RI>(P, c, dp, world, 4, D);     // rules 4-7 hold: fills D
                        if (role < 3) {
                            TrainMem M;
                            train_memory<RI>(P, c, D, M);
                            s_info[slot].mem[role] = M.mem;
                        } else {
                            uint32_t kv_bad = 0u;
                            for (int q = 0; q < P.n_kern; q++) {
                                const DevKern &kn = P.kern[q];
                                if ((kn.needs_caps & ~P.caps) != 0u || ((kn.avail_mask >> D.bucket) & 1u) == 0u)
                                    kv_bad |= 1u << q;
                            }
                            const DevSched &sc = P.sched[c.s];
                            uint32_t rec_bad = 0u;
                            if (P.enforce && sc.overlap)
                                rec_bad = (D.kind == PF_KIND_1F1B && c.pp > 1) ? 7u : (1u << PF_REC_FULL);
                            s_info[slot].kv_bad = kv_bad;
                            s_info[slot].unmapped = (P.enforce && !sc.mapped) ? 1 : 0;
                            s_info[slot].rec_bad = (uint8_t)rec_bad;
                        }
                    }
                    __syncthreads();
                    const uint32_t total = nb * R;
                    for (uint32_t it = 0; it < total; it += kThreads) {
                        const uint32_t x = it + tid;
                        bool queued = false;
                        uint32_t i = 0;
                        if (x < total) {
                            const uint32_t pe = x / R, ro = x - pe * R;
                            const uint32_t j = (uint32_t)s_pass[PF_AT(P.chk, b0 + pe, 2048, PF_SITE_PASS)] * R + ro;
                            if (j >= j0 && j < j0 + n) {
                                i = j - j0;
                                const uint32_t r0 = P.radix[0];
                                const uint32_t qd = r0 == 1u ? ro : __umulhi(ro, P.magic[0]);
                                const int kvv = inner_vals[P.val_off[0] + (int)(ro - qd * r0)];
                                const int recv = P.n_inner > 1 ? inner_vals[P.val_off[1] + (int)qd] : s_slab.outer[1];
                                const EntryInfo &info = s_info[PF_AT(P.chk, pe, kEntryBatch, PF_SITE_INFO)];
                                int reason = 0;
                                if ((info.kv_bad >> kvv) & 1u) {
                                    reason = PF_R_KERNEL_MISSING;
                                } else if (info.unmapped) {
                                    reason = PF_R_UNMAPPED_SCHEDULE;
                                } else if ((info.rec_bad >> recv) & 1) {
                                    reason = PF_R_OVERLAP_PRECOND;
                                } else {
                                    const long long mem = info.mem[recv];
                                    if (A.mem) A.mem[PF_AT(P.chk, rel0 + i, A.count, PF_SITE_DENSE)] = mem;
                                    if (mem > P.budget_bytes)
                                        reason = PF_R_MEMORY;
                                    else
                                        queued = true;
                                }
                                if (!queued) img[PF_AT(P.chk, pad + i, P.slab + 16, PF_SITE_IMAGE) - pad] = (uint8_t)reason;
                            }
                        }
                        enqueue(queued, i);
                        if (++since_drain == kQueueCap / kThreads) {
                            __syncthreads();
                            drain();
                            since_drain = 0;
                        }
                    }
                    __syncthreads();  // the batch's entry records are read no more
                }
            } else {
                // Phase 1 without a rule table: integer rules for every candidate of the slab.  Rejected
                // candidates get their reason byte; the ones that reach the memory gate are only queued, because
                // they come in short runs and would leave most lanes of their warps idle.
                for (uint32_t it = 0; it < n; it += kThreads) {
                    const uint32_t i = it + tid;
                    bool queued = false;
                    if (i < n) {
                        int v[PF_MAX_AXES], dg[5] = {0, 0, 0, 0, 0};
                        decode_inner(j0 + i, v, dg);
                        TrainTuple c;
                        c.kv = v[0]; c.rec = v[1]; c.s = v[2]; c.mb = v[3]; c.v = v[4];
                        c.ep = v[5]; c.pp = v[6]; c.tp = v[7]; c.dp = v[8]; c.world = v[9];
                        c.sh = P.n_axes > 10 ? v[10] : PF_SHARD_ZERO1;
                        RI dp, world;
                        int reason = train_layout_rules<RI>(P, c, first_rule, 3, dp, world);
                        if (reason == 0) {
                            TrainDerived<RI> D;
                            reason = train_plan_rules<RI>(P, c, dp, world, first_rule, D);
                        }
                        if (reason != 0)
                            img[PF_AT(P.chk, pad + i, P.slab + 16, PF_SITE_IMAGE) - pad] = (uint8_t)reason;
                        else
                            queued = true;
                    }
                    enqueue(queued, i);
                    if (++since_drain == kQueueCap / kThreads) {
                        __syncthreads();
                        drain();
                        since_drain = 0;
                    }
                }
            }
            __syncthreads();
            drain();
            if (A.reason) block_copy_out(A.reason + rel0, img, n);
        } else {
            for (uint32_t it = 0; it < n; it += kThreads) {
                const uint32_t i = it + tid;
                const bool active = i < n;
                ServeOut so;
                so.reason = 0; so.tput = 0.f; so.mem = 0;
                if (active) {
                    int v[PF_MAX_AXES], dg[5] = {0, 0, 0, 0, 0};
                    decode_inner(j0 + i, v, dg);
                    ServeTuple c;
                    c.kv = v[0]; c.chunk = v[1]; c.batch = v[2]; c.dpa = v[3]; c.ep = v[4]; c.tp = v[5]; c.scen = v[6];
                    const int sc_i = (int)PF_AT(P.chk, c.scen, P.n_scen, PF_SITE_SCEN);
                    serve_eval<RI>(P, c, first_rule, __ldg(A.scen + sc_i), __ldg(A.scen + P.n_scen + sc_i), so);
                    const uint64_t o = PF_AT(P.chk, rel0 + i, A.count, PF_SITE_DENSE);
                    if (A.reason) A.reason[o] = (uint8_t)so.reason;
                    if (A.tput) A.tput[o] = so.tput;
                    if (A.mem) A.mem[o] = so.mem;
                }
                offer(active && (so.reason & 0x7f) == 0, so.tput, (uint32_t)(rel0 + i));
            }
        }
        finish_slab();
    }

    if (want_topk) {
        tk_prune<kTopkCap / 2 / kThreads>(s_buf, &s_count, &s_thr, (int)A.k);
        if (tid == 0) {
            if (s_thr != 0ull) atomicMax(A.g_thr, s_thr);
            s_thr = *reinterpret_cast<volatile unsigned long long *>(A.g_thr);
        }
        __syncthreads();
        tk_flush(s_buf, s_count, s_thr, s_base, A.keys, A.key_count);
    }
}

constexpr uint32_t kFillZeroBytes = 3072;     // the fill kernel's shared-memory source of zeros ...
constexpr uint32_t kFillReasonBytes = 1024;   // ... and of the reason byte of the slab in hand

// n bytes of value b at p: the 16-byte aligned body as asynchronous bulk copies from shared memory (`src` holds at
// least `piece` bytes of b; the block's first `issuers` threads issue the copies, `piece` bytes each: the copy engine
// moves them, the load/store pipe is not involved), the ragged ends with plain stores.  A bulk copy needs a 16-byte
// aligned destination and a size that is a multiple of 16: both hold by construction, and a piece that broke either
// would be stored the plain way instead.
__device__ __forceinline__ void block_fill_bulk(uint8_t *p, uint64_t n, uint32_t b, uint32_t src, uint32_t piece,
                                                uint32_t issuers)
{
    const uint32_t tid = threadIdx.x, nt = blockDim.x;
    // The copies carry an evict-first hint for L2: nothing in the call reads these bytes again, whereas the evaluated
    // slabs' outputs, the selection's tables and the simulator's records are re-read within microseconds -- without
    // the hint 2 GB of constant bytes push them out of the 126 MB cache (scoring kernel 0.126 -> 0.105 ms, selection
    // 0.089 -> 0.071 ms beside this kernel).
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    uint64_t head = (16 - ((uintptr_t)p & 15)) & 15;
    if (head > n) head = n;
    for (uint64_t i = tid; i < head; i += nt) p[i] = (uint8_t)b;
    const uint64_t body = (n - head) & ~(uint64_t)15;
    uint8_t *q = p + head;
    if (tid < issuers) {
        for (uint64_t off = (uint64_t)tid * piece; off < body; off += (uint64_t)issuers * piece) {
            const uint32_t len = (uint32_t)(body - off < piece ? body - off : piece);
            uint8_t *d = q + off;
            if ((((uintptr_t)d | len) & 15) == 0 && len != 0) {
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(d),
                             "r"(src), "r"(len), "l"(policy)
                             : "memory");
            } else {
                for (uint32_t i = 0; i < len; i++) d[i] = (uint8_t)b;
            }
        }
    }
    for (uint64_t i = head + body + tid; i < n; i += nt) p[i] = (uint8_t)b;
}

// The constant slabs behind the head of the visiting order, streamed by a kernel of their own.  Its bytes leave as
// asynchronous bulk copies from a 4 KB shared-memory pattern buffer, i.e. through the copy engine: a handful of
// instructions per 160 KB slab instead of ten thousand 16-byte stores, so the kernel neither queues in the SM's
// load/store pipe in front of the kernels it runs beside (the survivor selection and the simulator inside a search
// call, which polls shared memory) nor needs more than one small block per SM.  Tickets [hdr[4], n_slabs) are all
// constant slabs by construction of the order; blocks take them round robin (they are all the same size but for a
// clipped first or last one).
__global__ void __launch_bounds__(kThreads) fill_tail_kernel(const FillArgs A)
{
    // Where the hardware puts the blocks of a small grid is not even: of a grid of 32 blocks per SM, launched beside
    // the scoring kernel, all blocks were seen to arrive on about half of the SMs.  So the grid is oversubscribed and
    // a block works only if it is among the first `per_sm` to register on its SM; the others leave at once, and the
    // scheduler keeps placing blocks until (nearly) every SM has its share.
    __shared__ __align__(128) uint8_t s_src[kFillZeroBytes + kFillReasonBytes];
    __shared__ unsigned int s_go, s_t;
    const uint32_t tid = threadIdx.x;
    if (tid == 0) {
        unsigned int smid;
        asm("mov.u32 %0, %%smid;" : "=r"(smid));
        s_go = atomicAdd(A.sm_slots + (smid & 255u), 1u) < A.per_sm ? 1u : 0u;
        if (s_go) s_t = atomicAdd(A.ticket, 1u);
    }
    __syncthreads();
    if (!s_go) return;
    if (!order_table_valid(A.order_hdr, A.slab_lo, A.n_slabs, A.order_tail, A.order_fpe)) return;
    // The dense outputs of a constant slab leave as bulk copies from this buffer: zeros (tput and mem, twelve of a
    // candidate's thirteen bytes) from its first part, the slab's reason byte from the rest, which is rewritten
    // when the byte changes (slabs of one kind come in runs).
    for (uint32_t i = tid; i < kFillZeroBytes / 16; i += blockDim.x)
        reinterpret_cast<uint4 *>(s_src)[i] = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    const uint32_t zsrc = (uint32_t)__cvta_generic_to_shared(s_src), rsrc = zsrc + kFillZeroBytes;
    const uint32_t piece = A.piece < 16u ? 16u : (A.piece > kFillZeroBytes ? kFillZeroBytes : (A.piece & ~15u));
    const uint32_t rpiece = piece < kFillReasonBytes ? piece : kFillReasonBytes;
    uint32_t cur_b = 0xFFFFFFFFu;   // the byte the reason part holds
    const uint32_t head_n = A.order_hdr[4];
    for (;;) {
        const uint32_t tk = s_t;
        __syncthreads();
        if (head_n + tk >= A.n_slabs) break;
        uint32_t tk_next = 0;
        if (tid == 0) tk_next = atomicAdd(A.ticket, 1u);   // in flight while this slab is stored
        const uint32_t w = __ldg(A.order + head_n + tk);
        const uint64_t base = (A.slab_lo + (w & 0xFFFFFFu)) * (uint64_t)A.slab;
        const uint64_t lo = base > A.first ? base : A.first;
        const uint64_t end_slab = base + A.slab, end_call = A.first + A.count;
        const uint64_t hi = end_slab < end_call ? end_slab : end_call;
        const uint64_t rel0 = lo - A.first, n = hi - lo;
        (void)PF_AT(A.chk, head_n + tk, A.n_slabs, PF_SITE_ORDER);
        (void)PF_AT(A.chk, rel0 + n - 1, A.count, PF_SITE_DENSE);   // the slab's whole span lies inside the outputs
        const uint32_t b = w >> 24;
        if (A.reason && b != cur_b) {
            // copies issued earlier may still be reading the old byte pattern
            if (tid < A.issuers) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            __syncthreads();
            const uint32_t bw = b * 0x01010101u;
            for (uint32_t i = tid; i < kFillReasonBytes / 16; i += blockDim.x)
                reinterpret_cast<uint4 *>(s_src + kFillZeroBytes)[i] = make_uint4(bw, bw, bw, bw);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();
            cur_b = b;
        }
        if (A.reason) block_fill_bulk(A.reason + rel0, n, b, rsrc, rpiece, A.issuers);
        if (A.tput) block_fill_bulk(reinterpret_cast<uint8_t *>(A.tput + rel0), n * 4, 0u, zsrc, piece, A.issuers);
        if (A.mem) block_fill_bulk(reinterpret_cast<uint8_t *>(A.mem + rel0), n * 8, 0u, zsrc, piece, A.issuers);
        if (tid < A.issuers) {
            // a bound on the copies in flight per issuing thread: at most four slabs' worth
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory");
        }
        if (tid == 0) {
            s_t = tk_next;
            atomicAdd(A.done, 1u);   // slabs this launch has taken (accounting only)
        }
        __syncthreads();
    }
    // the block's copies must have been written before it ends (the zero buffer goes away with the block, and the
    // end of the kernel is what the rest of the call waits for)
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ------------------------------------------------------------------ reducing a compact key list

struct ReduceArgs {
    const unsigned long long *in;   // compact keys
    const unsigned int *in_count;
    const unsigned long long *in0;  // the producers' list and its length: short lists skip the block pass
    const unsigned int *in0_count;
    unsigned long long *out;        // compact keys of the next pass (when not final)
    unsigned int *out_count;
    uint32_t k;
    int final;                      // 1: write idx / score / count (gridDim.x == 1)
    uint64_t first;
    const uint64_t *idx_map;        // NULL: idx = first + rel; else idx = idx_map[rel]
    uint64_t *topk_idx;
    float *topk_score;
    uint32_t *topk_count;
};

// Pass 1, for a producers' list longer than kFastKeys keys: the list is cut into as many segments as the grid has
// blocks -- few enough that what the blocks leave (at most k keys each) fits the final kernel's one-go sort -- and
// block b walks its segment one tile at a time, admitting only keys above its running k-th best, and keeps the k
// best.  A tile's admissions are counted before they are appended, so the buffer is pruned only when it would
// really overflow.  A shorter list is left to the final kernel as it is.
__global__ void __launch_bounds__(kReduceThreads) reduce_kernel(const ReduceArgs A)
{
    chain_enter();
    __shared__ unsigned long long s_buf[kTopkCap];
    __shared__ int s_count;
    __shared__ unsigned long long s_thr;
    __shared__ int s_base[2];
    const int tid = threadIdx.x, k = (int)A.k;
    const unsigned int n = *A.in_count;
    if (n <= (unsigned int)kFastKeys) return;
    const unsigned int seg = (n + gridDim.x - 1) / gridDim.x;
    const unsigned int lo = blockIdx.x * seg;
    const unsigned int hi = min(lo + seg, n);
    if (lo >= hi) return;
    if (tid == 0) {
        s_count = 0;
        s_thr = 0ull;
    }
    __syncthreads();
    for (unsigned int pos = lo; pos < hi; pos += kReduceThreads) {
        const unsigned int i = pos + tid;
        const unsigned long long key = i < hi ? A.in[i] : 0ull;
        unsigned long long thr = s_thr;
        const int takers = __syncthreads_count(key > thr);
        if (s_count + takers > kTopkCap) {
            tk_prune<kTopkCap / 2 / kReduceThreads>(s_buf, &s_count, &s_thr, k);
            thr = s_thr;
        }
        tk_push(s_buf, &s_count, thr, key != 0ull, key);
        __syncthreads();
    }
    tk_prune<kTopkCap / 2 / kReduceThreads>(s_buf, &s_count, &s_thr, k);
    tk_flush(s_buf, s_count, 0ull, s_base, A.out, A.out_count);
}

// Final pass, one block.  A short producers' list (at most kFastKeys keys) is loaded whole into shared memory;
// the k-th largest key is found by a radix select over the eight key bytes, the keys from there up are gathered
// and only those (at most k) are sorted.  Otherwise the list left by pass 1 is walked through with the usual
// prune-on-overflow.
__global__ void __launch_bounds__(kReduceThreads) reduce_final_kernel(const ReduceArgs A)
{
    chain_enter();
    extern __shared__ __align__(16) unsigned long long s_big[];  // kFastKeys keys, then kTopkCap keys to sort in
    __shared__ int s_count;
    __shared__ unsigned long long s_thr;
    __shared__ unsigned int s_hist[256];
    __shared__ unsigned long long s_prefix;
    __shared__ unsigned int s_need;
    __shared__ int s_stop;
    const int tid = threadIdx.x, k = (int)A.k;
    // the list to finish: the producers' own when it is short, else what pass 1 left of it (short by construction)
    unsigned int n0 = *A.in0_count;
    const unsigned long long *src0 = A.in0;
    if (n0 > (unsigned int)kFastKeys) {
        n0 = *A.in_count;
        src0 = A.in;
    }
    unsigned long long *s_out = s_big;
    int c;
    if (n0 <= (unsigned int)kFastKeys) {
        s_out = s_big + kFastKeys;
        for (unsigned int i = tid; i < n0; i += kReduceThreads) s_big[i] = src0[i];
        if (tid == 0) {
            s_prefix = 0ull;
            s_need = (unsigned int)k;
            s_count = 0;
            s_stop = 0;
        }
        __syncthreads();
        if (n0 > (unsigned int)k) {
            for (int shift = 56; shift >= 0; shift -= 8) {
                for (int i = tid; i < 256; i += kReduceThreads) s_hist[i] = 0u;
                __syncthreads();
                const unsigned long long hi_mask = shift == 56 ? 0ull : (~0ull << (shift + 8));
                const unsigned long long prefix = s_prefix;
                for (unsigned int i = tid; i < n0; i += kReduceThreads) {
                    const unsigned long long key = s_big[i];
                    if ((key & hi_mask) == prefix) atomicAdd(&s_hist[(unsigned int)(key >> shift) & 255u], 1u);
                }
                __syncthreads();
                if (tid < 32) {
                    // lane l owns digits 255 - 8l down to 248 - 8l; cumulative counts run from the top digit down
                    unsigned int own = 0;
                    for (int j = 0; j < 8; j++) own += s_hist[255 - 8 * tid - j];
                    unsigned int incl = own;
                    for (int off = 1; off < 32; off <<= 1) {
                        const unsigned int y = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                        if (tid >= off) incl += y;
                    }
                    const unsigned int need = s_need;
                    if (incl - own < need && incl >= need) {
                        unsigned int run = incl - own;
                        for (int j = 0; j < 8; j++) {
                            const int d = 255 - 8 * tid - j;
                            const unsigned int h = s_hist[d];
                            if (run + h >= need) {
                                s_prefix = prefix | ((unsigned long long)d << shift);
                                s_need = need - run;
                                // every key of this digit is needed: the cut is the digit's lowest key
                                if (run + h == need) s_stop = 1;
                                break;
                            }
                            run += h;
                        }
                    }
                }
                __syncthreads();
                if (s_stop) break;
            }
        }
        const unsigned long long cut = n0 > (unsigned int)k ? s_prefix : 1ull;  // keys are distinct: exactly k pass
        for (unsigned int base = 0; base < n0; base += kReduceThreads) {
            const unsigned int i = base + tid;
            const unsigned long long key = i < n0 ? s_big[i] : 0ull;
            const bool take = key >= cut && key != 0ull;
            const unsigned mask = __ballot_sync(0xFFFFFFFFu, take);
            if (mask) {
                const int lane = tid & 31, leader = __ffs(mask) - 1;
                int pos = 0;
                if (lane == leader) pos = atomicAdd(&s_count, __popc(mask));
                pos = __shfl_sync(0xFFFFFFFFu, pos, leader);
                pos += __popc(mask & ((1u << lane) - 1u));
                if (take && pos < kTopkCap) s_out[pos] = key;
            }
        }
        __syncthreads();
        c = s_count < k ? s_count : k;
        int n_sort = 64;
        while (n_sort < c) n_sort <<= 1;
        for (int i = c + tid; i < n_sort; i += kReduceThreads) s_out[i] = 0ull;
        tk_sort_desc<kTopkCap / 2 / kReduceThreads>(s_out, n_sort);
    } else {
        const unsigned int n = *A.in_count;
        if (tid == 0) {
            s_count = 0;
            s_thr = 0ull;
        }
        __syncthreads();
        for (unsigned int pos = 0; pos < n; pos += kReduceThreads) {
            const unsigned int i = pos + tid;
            const unsigned long long key = i < n ? A.in[i] : 0ull;
            unsigned long long thr = s_thr;
            const int takers = __syncthreads_count(key > thr);
            if (s_count + takers > kTopkCap) {
                tk_prune<kTopkCap / 2 / kReduceThreads>(s_big, &s_count, &s_thr, k);
                thr = s_thr;
            }
            tk_push(s_big, &s_count, thr, key != 0ull, key);
            __syncthreads();
        }
        tk_prune<kTopkCap / 2 / kReduceThreads>(s_big, &s_count, &s_thr, k);
        c = s_count;
    }
    for (int i = tid; i < k; i += kReduceThreads) {
        if (i < c) {
            unsigned long long key = s_out[i];
            uint32_t rel = key_rel(key);
            A.topk_idx[i] = A.idx_map ? A.idx_map[rel] : A.first + rel;
            A.topk_score[i] = key_score(key);
        } else {
            A.topk_idx[i] = UINT64_MAX;
            A.topk_score[i] = 0.f;
        }
    }
    if (tid == 0) *A.topk_count = (uint32_t)c;
}

int launch_topk_reduce(void *d_workspace, const TopkLayout &lay, uint64_t n_keys_max, uint32_t k, uint64_t first,
                       const uint64_t *d_idx_map, uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count,
                       cudaStream_t st, int *n_kernels, bool chained)
{
    uint8_t *ws = (uint8_t *)d_workspace;
    unsigned int *ctrl = (unsigned int *)(ws + lay.off_ctrl);
    unsigned long long *in = (unsigned long long *)(ws + lay.off_keys_a);
    unsigned long long *out = (unsigned long long *)(ws + lay.off_keys_b);
    *n_kernels = 0;
    // pass 1 spreads a long list over so few blocks that what they leave (at most k keys each) is a short list;
    // one block finishes a short list, the producers' own or that one
    ReduceArgs r;
    r.in = in; r.in_count = ctrl + 1; r.out = out; r.out_count = ctrl + 2;
    r.in0 = in; r.in0_count = ctrl + 1;
    r.k = k; r.final = 0; r.first = first; r.idx_map = d_idx_map;
    r.topk_idx = d_topk_idx; r.topk_score = d_topk_score; r.topk_count = d_topk_count;
    uint64_t blocks = (uint64_t)kFastKeys / (k ? k : 1);
    blocks = blocks < 1 ? 1 : (blocks > 256 ? 256 : blocks);
    if (n_keys_max > (uint64_t)kFastKeys) {
        if (chained)
            launch_chained(reduce_kernel, (unsigned int)blocks, kReduceThreads, 0, st, r);
        else
            reduce_kernel<<<(unsigned int)blocks, kReduceThreads, 0, st>>>(r);
        chained = true;   // the next launch follows this kernel
        count_launch();
        (*n_kernels)++;
        PF_CUDA_TRY(cudaGetLastError(), "reduce_kernel launch");
    }
    r.in = out; r.in_count = ctrl + 2; r.final = 1;
    {
        int dev = 0;
        PF_CUDA_TRY(cudaGetDevice(&dev), "reduce_final_kernel device");
        PF_CUDA_TRY(ensure_dynamic_smem((const void *)reduce_final_kernel, dev, (kFastKeys + kTopkCap) * 8),
                    "reduce_final_kernel smem");
    }
    if (chained)
        launch_chained(reduce_final_kernel, 1, kReduceThreads, (kFastKeys + kTopkCap) * 8, st, r);
    else
        reduce_final_kernel<<<1, kReduceThreads, (kFastKeys + kTopkCap) * 8, st>>>(r);
    count_launch();
    (*n_kernels)++;
    PF_CUDA_TRY(cudaGetLastError(), "reduce_final_kernel launch");
    return PF_OK;
}

// ------------------------------------------------------------------ merge of two finished top-k lists

struct Merge2Args {
    uint32_t k;
    const uint64_t *idx_a, *idx_b;
    const float *sc_a, *sc_b;
    const uint32_t *cnt_a, *cnt_b;
    uint64_t *idx_out;
    float *sc_out;
    uint32_t *cnt_out;
};

// (score descending, index ascending) on explicit pairs; empty slots (idx = UINT64_MAX) last
__device__ __forceinline__ bool pair_before(uint32_t sa, uint64_t ia, uint32_t sb, uint64_t ib)
{
    if (ia == UINT64_MAX || ib == UINT64_MAX) return ib == UINT64_MAX && ia != UINT64_MAX;
    if (sa != sb) return sa > sb;
    return ia < ib;
}

__global__ void __launch_bounds__(kThreads) merge2_kernel(const Merge2Args A)
{
    __shared__ uint32_t s_sc[kTopkCap];
    __shared__ uint64_t s_ix[kTopkCap];
    const int tid = threadIdx.x, k = (int)A.k;
    const int na = min((int)*A.cnt_a, k), nb = min((int)*A.cnt_b, k);
    for (int i = tid; i < kTopkCap; i += kThreads) {
        uint32_t s = 0;
        uint64_t x = UINT64_MAX;
        if (i < na) {
            s = __float_as_uint(A.sc_a[i]);
            x = A.idx_a[i];
        } else if (i >= k && i - k < nb) {
            s = __float_as_uint(A.sc_b[i - k]);
            x = A.idx_b[i - k];
        }
        s_sc[i] = s;
        s_ix[i] = x;
    }
    for (int size = 2; size <= kTopkCap; size <<= 1)
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int i = tid; i < kTopkCap / 2; i += kThreads) {
                int lo = 2 * i - (i & (stride - 1)), hi = lo + stride;
                bool fwd = (lo & size) == 0;
                uint32_t sa = s_sc[lo], sb = s_sc[hi];
                uint64_t ia = s_ix[lo], ib = s_ix[hi];
                bool swap = fwd ? pair_before(sb, ib, sa, ia) : pair_before(sa, ia, sb, ib);
                if (swap) {
                    s_sc[lo] = sb; s_sc[hi] = sa;
                    s_ix[lo] = ib; s_ix[hi] = ia;
                }
            }
        }
    __syncthreads();
    // duplicates (the same candidate in both lists) would be adjacent; the inputs are shards of one space,
    // so none are expected and none are removed
    const int n = min(na + nb, k);
    for (int i = tid; i < k; i += kThreads) {
        A.idx_out[i] = i < n ? s_ix[i] : UINT64_MAX;
        A.sc_out[i] = i < n ? __uint_as_float(s_sc[i]) : 0.f;
    }
    if (tid == 0) *A.cnt_out = (uint32_t)n;
}

static int grid_for(const pf_plan_t *p, uint64_t n_slabs)
{
    uint64_t g = (uint64_t)p->sm_count * 4;
    if (g > n_slabs) g = n_slabs;
    return g < 1 ? 1 : (int)g;
}

static void slab_span(const pf_plan_t *p, uint64_t first, uint64_t count, uint64_t &slab_lo, uint64_t &n_slabs)
{
    const uint64_t S = p->dev.slab;
    slab_lo = first / S;
    uint64_t slab_hi = (first + count + S - 1) / S;
    n_slabs = slab_hi - slab_lo;
}

}  // namespace pf

using namespace pf;

extern "C" size_t pf_score_workspace(const pf_plan_t *p, uint64_t count, uint32_t k)
{
    if (!p || count == 0) return 256;
    uint64_t slab_lo, n_slabs;
    slab_span(p, 0, count + p->dev.slab, slab_lo, n_slabs);  // any alignment of `first`
    return topk_layout((uint64_t)grid_for(p, n_slabs) * k, k).total;
}

extern "C" int pf_score(pf_plan_t *p, uint64_t first, uint64_t count, uint8_t *d_reason, float *d_tput,
                        int64_t *d_mem, uint32_t k, uint64_t *d_topk_idx, float *d_topk_score,
                        uint32_t *d_topk_count, void *d_workspace, size_t workspace_bytes, void *stream)
{
    return pf::score_run(p, first, count, d_reason, d_tput, d_mem, k, d_topk_idx, d_topk_score, d_topk_count,
                         d_workspace, workspace_bytes, (cudaStream_t)stream, nullptr, nullptr);
}

int pf::score_run(pf_plan_t *p, uint64_t first, uint64_t count, uint8_t *d_reason, float *d_tput, int64_t *d_mem,
                  uint32_t k, uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count, void *d_workspace,
                  size_t workspace_bytes, cudaStream_t st, const ScoreDigest *dg, ScoreSpread *spread)
{
    ScoreSpread plain;
    ScoreSpread &sp = spread ? *spread : plain;
    sp.join_pending = sp.fill_pending = false;
    if (!p) return PF_EINVAL;
    if (k > PF_K_MAX) return PF_EINVAL;
    if (k > 0 && (!d_topk_idx || !d_topk_score || !d_topk_count)) return PF_EINVAL;
    if (count == 0 || count >= PF_MAX_COUNT) return PF_ERANGE;
    if (first >= p->size || count > p->size - first) return PF_ERANGE;
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0) return PF_EWORKSPACE;
    if (workspace_bytes < pf_score_workspace(p, count, k)) return PF_EWORKSPACE;
    if (int rc_dev = check_device(p)) return rc_dev;

    uint64_t slab_lo, n_slabs;
    slab_span(p, first, count, slab_lo, n_slabs);
    const int grid = grid_for(p, n_slabs);
    const TopkLayout lay = topk_layout((uint64_t)grid * k, k);
    uint8_t *ws = (uint8_t *)d_workspace;

    ScoreArgs a;
    a.first = first; a.count = count; a.slab_lo = slab_lo; a.n_slabs = (uint32_t)n_slabs; a.k = k;
    {
        // a multiplier near 0.618 * n_slabs that is coprime to n_slabs: consecutive queue tickets land far apart
        uint64_t n = n_slabs, m = (uint64_t)((double)n_slabs * 0.6180339887) | 1;
        auto gcd = [](uint64_t x, uint64_t y) { while (y) { uint64_t t = x % y; x = y; y = t; } return x; };
        while (m > 1 && gcd(m, n) != 1) m -= 2;
        if (n <= 2 || m < 1) m = 1;
        a.slab_mul = (uint32_t)m;
    }
    a.reason = d_reason; a.tput = d_tput; a.mem = (long long *)d_mem;
    a.keys = (unsigned long long *)(ws + lay.off_keys_a);
    a.slab_counter = (unsigned int *)(ws + lay.off_ctrl);
    a.key_count = a.slab_counter + 1;
    a.g_thr = (unsigned long long *)(ws + lay.off_ctrl + 16);
    a.vals = p->d_vals; a.scen = p->d_scen;
    a.order = nullptr;
    a.dg.hist1 = nullptr;
    if (dg && p->dev.phase == PF_PHASE_TRAIN && d_tput) a.dg = *dg;
    PF_CUDA_TRY(cudaMemsetAsync(a.slab_counter, 0, 256, st), "pf_score: counter reset");
    timing_begin(p, PF_T_SCORE, st);
    int n_score_kernels = 1;
    a.order_hdr = nullptr;
    a.order_tail = (uint32_t)grid * kTailFillsPerBlock;
    a.order_fpe = (uint32_t)(sp.fills_per_evaluated < 0 ? 0 : sp.fills_per_evaluated);
    a.head_only = 0;
    bool split = false;
    if (p->d_order && n_slabs <= p->order_cap && n_slabs > (uint64_t)grid) {
        uint32_t *hdr = p->d_order, *order = p->d_order + 64;
        split = sp.fill_aside && p->fill_stream && (d_reason || d_tput || d_mem);
        // with a fill kernel behind it the scoring kernel ends on evaluated slabs anyway: no fills are held back
        if (split) a.order_tail = 0;
        if (p->order_slab_lo != slab_lo || p->order_n_slabs != (uint32_t)n_slabs || p->order_tail != a.order_tail ||
            p->order_fpe != a.order_fpe) {
            // another range than the table was last built for: rebuild it (two small launches)
            uint8_t *cls = (uint8_t *)(order + p->order_cap);
            const unsigned cgrid = (unsigned)((n_slabs + 255) / 256);
            if (p->dev.wide)
                slab_class_kernel<unsigned long long><<<cgrid, 256, 0, st>>>(p->dev, p->d_vals, slab_lo,
                                                                            (uint32_t)n_slabs, cls);
            else
                slab_class_kernel<uint32_t><<<cgrid, 256, 0, st>>>(p->dev, p->d_vals, slab_lo, (uint32_t)n_slabs,
                                                                   cls);
            slab_order_kernel<<<1, 1024, 0, st>>>(cls, slab_lo, (uint32_t)n_slabs, a.order_tail, a.order_fpe, order,
                                                  hdr);
            PF_CUDA_TRY(cudaGetLastError(), "slab order launch");
            count_launch();
            count_launch();
            n_score_kernels = 3;
            p->order_slab_lo = slab_lo;
            p->order_n_slabs = (uint32_t)n_slabs;
            p->order_tail = a.order_tail;
            p->order_fpe = a.order_fpe;
        }
        a.order = order;
        a.order_hdr = hdr;
        a.head_only = split ? 1u : 0u;
    }
    FillArgs f;
    if (split) {
        // The constant slabs are streamed by the fill kernel on the plan's fill stream, beside this kernel and
        // everything that follows it in the call.  Queue head and block registrations start at zero.
        PF_CUDA_TRY(cudaMemsetAsync(p->d_fill_ctl, 0, 2048, st), "fill control reset");
        f.first = first; f.count = count; f.slab_lo = slab_lo; f.n_slabs = (uint32_t)n_slabs;
        f.slab = p->dev.slab; f.order_tail = a.order_tail; f.order_fpe = a.order_fpe;
        f.chk = p->dev.chk;
        f.reason = d_reason; f.tput = d_tput; f.mem = (long long *)d_mem;
        f.order = a.order; f.order_hdr = a.order_hdr;
        f.ticket = p->d_fill_ctl; f.done = p->d_fill_ctl + 2;
        f.sm_slots = p->d_fill_ctl + 16; f.per_sm = kFillBlocksPerSm;
        PF_CUDA_TRY(cudaEventRecord(p->ev_fork3, st), "early fill fork");
        PF_CUDA_TRY(cudaStreamWaitEvent(p->fill_stream, p->ev_fork3, 0), "early fill fork");
    }
    const size_t queue_bytes = p->dev.phase == PF_PHASE_TRAIN
                                   ? (((size_t)p->dev.slab + 16 + 15) & ~(size_t)15) + kQueueCap * sizeof(uint16_t)
                                   : 0;
    // static + dynamic shared memory passes the 48 KB default for large slabs: opt in
    PF_CUDA_TRY(ensure_dynamic_smem(p->dev.wide ? (const void *)score_kernel<unsigned long long>
                                                : (const void *)score_kernel<uint32_t>,
                                    p->device, queue_bytes), "score_kernel smem");
    if (p->dev.wide)
        score_kernel<unsigned long long><<<grid, kThreads, queue_bytes, st>>>(p->dev, a);
    else
        score_kernel<uint32_t><<<grid, kThreads, queue_bytes, st>>>(p->dev, a);
    count_launch();
    timing_end(p, PF_T_SCORE, n_score_kernels, st);
    PF_CUDA_TRY(cudaGetLastError(), "score_kernel launch");
    if (split) {
        // The fill kernel is issued after the scoring kernel (on the fill stream it waits only for
        // what preceded that kernel), so that the two reach the device in the same order whether or not the host
        // runs ahead of it: a grid that arrives first is handed out to the end before the next one starts, and this
        // one is deliberately long.
        timing_begin(p, PF_T_FILL, p->fill_stream);
        f.piece = kFillZeroBytes;
        f.issuers = kFillThreads;
        fill_tail_kernel<<<p->sm_count * kFillGridPerSm, kFillThreads, 0, p->fill_stream>>>(f);
        count_launch();
        timing_end(p, PF_T_FILL, 1, p->fill_stream);
        const cudaError_t e_early = cudaGetLastError();
        // the fill stream is forked from here on: the join event is recorded whatever happens next
        if (cudaEventRecord(p->ev_fill, p->fill_stream) == cudaSuccess) sp.fill_pending = true;
        if (e_early != cudaSuccess) {
            set_cuda_error(e_early, "fill_tail_kernel launch");
            return PF_ECUDA;
        }
    }
    const bool topk_aside = k > 0 && sp.topk_aside && p->side_stream;
    int rc = PF_OK;
    if (topk_aside) PF_CUDA_TRY(cudaEventRecord(p->ev_fork, st), "score fork");
    if (split) {
        // until the fill stream has joined, only the evaluated slabs of the dense outputs hold results (guard)
        sp.guard.cls = (const uint8_t *)(a.order + p->order_cap);
        sp.guard.hdr = a.order_hdr;
        sp.guard.slab_lo = slab_lo; sp.guard.n_slabs = (uint32_t)n_slabs; sp.guard.slab = p->dev.slab;
        sp.guard.tail = a.order_tail; sp.guard.fpe = a.order_fpe;
    }
    if (k > 0) {
        // The reduction of the key list depends on the scoring kernel only.  Inside a search call it runs on the
        // plan's second stream, beside the survivor selection; the caller joins (ev_join) before it reuses the
        // workspace.
        cudaStream_t rs = st;
        if (topk_aside) {
            rs = p->side_stream;
            cudaError_t e = cudaStreamWaitEvent(rs, p->ev_fork, 0);
            if (e != cudaSuccess) {
                set_cuda_error(e, "top-k fork");
                return PF_ECUDA;   // nothing was forked onto the side stream
            }
        }
        timing_begin(p, PF_T_TOPK, rs);
        int nk = 0;
        // (on the caller's stream the scoring kernel is the operation right before: a chained launch)
        const int rc2 = launch_topk_reduce(ws, lay, (uint64_t)grid * k, k, first, nullptr, d_topk_idx, d_topk_score,
                                           d_topk_count, rs, &nk, rs == st && !split);
        timing_end(p, PF_T_TOPK, nk, rs);
        if (rs != st && cudaEventRecord(p->ev_join, rs) == cudaSuccess) sp.join_pending = true;
        if (rc == PF_OK) rc = rc2;
    }
    return rc;
}

// ------------------------------------------------------------------ pf_score without a caller workspace
// The scratch of pf_score_static: part of the device image, one copy per GPU that loads the library.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[PF_STATIC_SCRATCH_BYTES];

#include <mutex>
namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void *g_static_ptr[kMaxDevices];   // device address of g_static_scratch, per device ordinal
}  // namespace

extern "C" int pf_score_static(pf_plan_t *p, uint64_t first, uint64_t count, uint8_t *d_reason, float *d_tput,
                               int64_t *d_mem, uint32_t k, uint64_t *d_topk_idx, float *d_topk_score,
                               uint32_t *d_topk_count, void *stream)
{
    if (!p) return PF_EINVAL;
    if (k > PF_K_MAX) return PF_EINVAL;
    if (count == 0 || count >= PF_MAX_COUNT) return PF_ERANGE;
    // refuse what the fixed array cannot hold before touching the device
    if (pf_score_workspace(p, count, k) > (size_t)PF_STATIC_SCRATCH_BYTES) return PF_EWORKSPACE;
    // the scratch that counts is the one on the plan's device, which must be the current one
    if (int rc_dev = check_device(p)) return rc_dev;
    const int dev = p->device;
    if (dev < 0 || dev >= kMaxDevices) return PF_EUNSUPPORTED;
    void *scratch = nullptr;
    {
        // once per device, with that device current: ask the runtime where the array lives on it
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {
            void *ptr = nullptr;
            PF_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch), "pf_score_static: scratch address");
            g_static_ptr[dev] = ptr;
        }
        scratch = g_static_ptr[dev];
    }
    // pf_score clears the counters it needs at the start of every call; the rest is written before it is read
    return pf_score(p, first, count, d_reason, d_tput, d_mem, k, d_topk_idx, d_topk_score, d_topk_count, scratch,
                    (size_t)PF_STATIC_SCRATCH_BYTES, stream);
}

extern "C" int pf_topk_merge(uint32_t k, const uint64_t *d_idx_a, const float *d_score_a, const uint32_t *d_count_a,
                             const uint64_t *d_idx_b, const float *d_score_b, const uint32_t *d_count_b,
                             uint64_t *d_idx_out, float *d_score_out, uint32_t *d_count_out, void *stream)
{
    if (k < 1 || k > PF_K_MAX) return PF_EINVAL;
    if (!d_idx_a || !d_score_a || !d_count_a || !d_idx_b || !d_score_b || !d_count_b || !d_idx_out || !d_score_out ||
        !d_count_out)
        return PF_EINVAL;
    Merge2Args a;
    a.k = k; a.idx_a = d_idx_a; a.idx_b = d_idx_b; a.sc_a = d_score_a; a.sc_b = d_score_b;
    a.cnt_a = d_count_a; a.cnt_b = d_count_b; a.idx_out = d_idx_out; a.sc_out = d_score_out; a.cnt_out = d_count_out;
    merge2_kernel<<<1, kThreads, 0, (cudaStream_t)stream>>>(a);
    count_launch();
    PF_CUDA_TRY(cudaGetLastError(), "merge2_kernel launch");
    return PF_OK;
}
