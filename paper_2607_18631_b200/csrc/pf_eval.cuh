// pf_eval.cuh -- per-candidate evaluation on the device: realizability rules (integers), memory model
// (int64), analytic step time and pricing (fp32).  Used by the scoring kernel and by the simulator kernel
// (which needs the same per-layer terms).  Follows the predicate's fixed order (Sec. 3.3, Fig. 2):
// structural checks, emit dry-run rules, memory gate; then the closed-form scorer (Sec. 3.2) and the
// realization tax, throughput / (1 + frac) (Sec. 3.2).
#pragma once

#include "pf_internal.cuh"

namespace pf {

typedef long long i64;

// ceil(a / b) for a >= 0, b >= 1.  Parallel degrees are almost always powers of two: those take a shift
// (the branch is uniform wherever the degree is, i.e. across a slab), anything else the 64-bit division.
__device__ __forceinline__ i64 cdiv64(i64 a, i64 b)
{
    if ((b & (b - 1)) == 0) return (a + b - 1) >> (63 - __clzll(b));
    return (a + b - 1) / b;
}

// fp32 quotient by reciprocal-multiply (2 ulp): the step-time model tolerates 1e-4 relative, and its ~20
// quotients per candidate are otherwise the largest block of instructions in the cost model
__device__ __forceinline__ float fdiv(float a, float b) { return __fdividef(a, b); }

// Which parts of the calibration domain a query falls outside of (PF_WHY_* bits); 0 inside or with no domain.
template <typename RI>
__device__ __forceinline__ uint32_t domain_why(const DevPlan &P, const DevKern &kn, RI m_e)
{
    if (!P.dom_attached) return 0u;
    uint32_t why = 0u;
    if (P.dom_gpu >= 0 && P.dom_gpu != P.gpu_id) why |= PF_WHY_GPU;
    if (((P.dom_dtypes >> kn.dtype) & 1u) == 0u) why |= PF_WHY_DTYPE;
    if ((i64)m_e < (i64)P.dom_m_lo) why |= PF_WHY_M_LOW;
    if ((i64)m_e > (i64)P.dom_m_hi) why |= PF_WHY_M_HIGH;
    return why;
}

// tokens-per-expert bucket over the calibration domain [64, 8192]: <128, 128.., 256.., ..., >= 8192
template <typename RI>
__device__ __forceinline__ int me_bucket(RI m_e)
{
    int hb = m_e == 0 ? 0 : (sizeof(RI) == 8 ? 63 - __clzll((long long)m_e) : 31 - __clz((int)m_e));
    int b = hb - 6;
    return b < 0 ? 0 : (b > 7 ? 7 : b);
}

struct Link {
    float bw, alpha;
};
__device__ __forceinline__ Link link_of(const DevPlan &P, i64 span)
{
    Link l;
    bool intra = span <= (i64)P.G;
    l.bw = intra ? P.bw_intra : P.bw_inter;
    l.alpha = intra ? P.alpha_intra : P.alpha_inter;
    return l;
}
__device__ __forceinline__ float ceil_log2f(i64 n) { return (float)(64 - __clzll(n - 1)); }  // n >= 2
// all-reduce (and reduce-scatter + all-gather): ring volume 2(n-1)/n, 2*ceil(log2 n) latency hops
__device__ __forceinline__ float t_allreduce(i64 n, float bytes, Link lk)
{
    if (n <= 1) return 0.f;
    float fn = (float)n;
    return fdiv(2.f * (fn - 1.f) * bytes, fn * lk.bw) + 2.f * ceil_log2f(n) * lk.alpha;
}
// all-gather of `bytes` (the gathered size); a reduce-scatter has the same form
__device__ __forceinline__ float t_allgather(i64 n, float bytes, Link lk)
{
    if (n <= 1) return 0.f;
    const float nf = (float)n;
    return fdiv((nf - 1.f) * bytes, nf * lk.bw) + ceil_log2f(n) * lk.alpha;
}
__device__ __forceinline__ float t_alltoall(i64 n, float bytes, Link lk)
{
    if (n <= 1) return 0.f;
    float fn = (float)n;
    return fdiv((fn - 1.f) * bytes, fn * lk.bw) + lk.alpha;
}

// ------------------------------------------------------------------ training

struct TrainTuple {
    int kv, rec, s, mb, v, ep, pp, tp, dp, world;  // dp / world as listed (0 = derived)
    int sh = PF_SHARD_ZERO1;                       // memory sharding (zero1 when the space has no such axis)
};

// Quantities the rules derive on the way, kept for the memory / time models and the simulator.
template <typename RI>
struct TrainDerived {
    RI dp, world, m, t, edp, m_e;
    int kind, ov, v_eff, Q, Lc, Ls, bucket;
    int nd0, nd_last;   // leading dense layers on the first rank and on the last one
};

// Rules first_rule..last_rule of the layout rules 1-3.  Returns 0 or the failing rule; fills dp / world.
template <typename RI>
__device__ __forceinline__ int train_layout_rules(const DevPlan &P, const TrainTuple &c, int first_rule, int last_rule,
                                                  RI &dp_out, RI &world_out)
{
    RI tp = (RI)c.tp, pp = (RI)c.pp, dp = (RI)c.dp, world = (RI)c.world;
    RI tppp = tp * pp;
    if (c.dp == 0) {
        RI q = world / tppp;
        if (first_rule <= 1 && q * tppp != world) return PF_R_WORLD;
        dp = q;
    }
    if (c.world == 0) world = tppp * dp;
    dp_out = dp;
    world_out = world;
    if (first_rule <= 1) {
        if (tppp * dp != world) return PF_R_WORLD;
        if (world < (RI)P.world_min || world > (RI)P.world_max) return PF_R_WORLD;
        if (world > (RI)P.G && world % (RI)P.G != 0) return PF_R_WORLD;
    }
    if (first_rule <= 2 && last_rule >= 2) {
        if (c.tp > P.tp_max || c.tp > P.G || P.nh % c.tp != 0) return PF_R_TP;
        if (P.S > 0 && P.Fs % c.tp != 0) return PF_R_TP;
        if (P.ep_scope == 0 && P.F % c.tp != 0) return PF_R_TP;
    }
    if (first_rule <= 3 && last_rule >= 3) {
        if (P.E % c.ep != 0) return PF_R_EP;
        RI group = P.ep_scope ? dp * tp : dp;
        if (group % (RI)c.ep != 0) return PF_R_EP;
    }
    return 0;
}

// Rules 4-10 (up to last_rule; rules 4-7 look at sched, mb, v and the layout only).  Returns 0 or the failing
// rule; fills D.
template <typename RI>
__device__ __forceinline__ int train_plan_rules(const DevPlan &P, const TrainTuple &c, RI dp, RI world, int first_rule,
                                                TrainDerived<RI> &D, int last_rule = 10)
{
    D.dp = dp;
    D.world = world;
    RI gbs = (RI)P.gbs;
    RI dpmb = dp * (RI)c.mb;
    RI m = gbs / dpmb;
    if (first_rule <= 4 && m * dpmb != gbs) return PF_R_BATCH;
    const DevSched &sc = P.sched[c.s];
    int kind = sc.kind;
    int v_eff = c.v == 0 ? (kind == PF_KIND_INTERLEAVED ? 2 : 1) : c.v;
    D.kind = kind;
    D.ov = sc.overlap;
    D.v_eff = v_eff;
    D.m = m;
    D.t = (RI)c.mb * (RI)P.seq;
    if (kind == PF_KIND_INTERLEAVED) {
        if (v_eff < 2 || c.pp < 2) return PF_R_VSTAGE;
    } else if (v_eff != 1) {
        return PF_R_VSTAGE;
    }
    // Q = pp * v_eff can exceed int only for absurd pp; the layer rule compares against L first
    long long Q64 = (long long)c.pp * v_eff;
    if (P.layer_mode == 0) {
        if (Q64 > P.L || P.L % (int)Q64 != 0) return PF_R_LAYERS;
    } else {
        if (Q64 > P.L) return PF_R_LAYERS;
    }
    int Q = (int)Q64;
    D.Q = Q;
    D.Lc = (P.L + Q - 1) / Q;
    D.Ls = v_eff * D.Lc;
    // Stage q covers layers [q Lc, (q+1) Lc) and rank r holds stages r, r + pp, ...: its chunks start every
    // pp Lc layers from layer r Lc.  Of the L_dense leading layers the rank's chunks before the last one reached are
    // dense throughout, that one as far as the dense layers go.
    D.nd0 = D.nd_last = 0;
    if (P.L_dense > 0) {
        const int stride = c.pp * D.Lc;
        auto dense_on_rank = [&](int first_layer) {
            const int left = P.L_dense - first_layer;          // dense layers from the rank's first chunk on
            if (left <= 0) return 0;
            const int whole = left / stride, rest = left - whole * stride;
            return whole >= v_eff ? v_eff * D.Lc : whole * D.Lc + min(rest, D.Lc);
        };
        D.nd0 = dense_on_rank(0);
        D.nd_last = dense_on_rank((c.pp - 1) * D.Lc);
    }
    if (kind == PF_KIND_INTERLEAVED) {
        if (m % (RI)c.pp != 0) return PF_R_MICROBATCH;
    } else if (kind == PF_KIND_DUALPIPE) {
        if ((m & 1) != 0) return PF_R_MICROBATCH;
        if (c.pp > 1 && (c.pp & 1) != 0) return PF_R_MICROBATCH;
    }
    if (last_rule < 8) return 0;
    RI tps = P.ep_scope ? (RI)c.tp : (RI)1;
    D.edp = P.ep_scope ? dp * (RI)c.tp / (RI)c.ep : dp / (RI)c.ep;
    D.m_e = (D.t * (RI)P.K * (RI)c.ep) / ((RI)P.E * tps);
    D.bucket = me_bucket<RI>(D.m_e);
    const DevKern &kn = P.kern[c.kv];
    if ((kn.needs_caps & ~P.caps) != 0u) return PF_R_KERNEL_MISSING;
    if (((kn.avail_mask >> D.bucket) & 1u) == 0u) return PF_R_KERNEL_MISSING;
    if (P.enforce) {
        if (!sc.mapped) return PF_R_UNMAPPED_SCHEDULE;
        if (sc.overlap && (c.rec == PF_REC_FULL || (kind == PF_KIND_1F1B && c.pp > 1))) return PF_R_OVERLAP_PRECOND;
    }
    return 0;
}

struct TrainMem {
    i64 N_dense, N_exp, n_shard, bytes_o, mem;
};

// Peak bytes on rank 0 (most in-flight activations): weights + gradients + sharded optimizer state
// (dense over dp, experts over the expert-DP group: Sec. 5 RQ1) + in-flight activations by schedule class.
template <typename RI>
__device__ __forceinline__ void train_memory(const DevPlan &P, const TrainTuple &c, const TrainDerived<RI> &D,
                                             TrainMem &M)
{
    const i64 tp = c.tp, pp = c.pp, t = (i64)D.t, m = (i64)D.m, Ls = D.Ls;
    const bool dual = D.kind == PF_KIND_DUALPIPE;
    const i64 copies = (dual && pp > 1) ? 2 : 1;
    const bool owns_head = (pp == 1) || dual;
    const i64 emb = cdiv64(P.P_emb, tp) * (owns_head ? 2 : 1);
    const i64 etp = P.ep_scope ? 1 : tp;
    // the rank's MoE layers (both stage copies of a DualPipe-style rank; the second copy sits at the far end of
    // the pipeline and has no leading dense layer) and its leading dense layers
    const i64 nd0 = D.nd0, n_moe = copies * Ls - nd0;
    M.N_dense = n_moe * (cdiv64(P.P_dl, tp) + P.P_rt) + emb;
    if (nd0) M.N_dense += nd0 * cdiv64(P.P_dld, tp);
    M.N_exp = n_moe * (i64)(P.E / c.ep) * cdiv64(P.P_e, etp);
    // parameters whose optimizer state this rank owns: dense over dp, experts over the expert-DP group
    M.n_shard = cdiv64(M.N_dense, (i64)D.dp) + cdiv64(M.N_exp, (i64)D.edp);
    // zero1: whole parameters and gradients, sharded state; offload: the state lives in host memory; fsdp:
    // parameters and gradients sharded like the state, plus the all-gather buffer of two layers' parameters
    i64 n_all = M.N_dense + M.N_exp, buf = 0;
    M.bytes_o = c.sh == PF_SHARD_ZERO1_OFFLOAD ? 0 : (i64)P.ob * M.n_shard;
    if (c.sh == PF_SHARD_FSDP) {
        n_all = M.n_shard;
        const i64 p_layer = cdiv64(P.P_dl, tp) + P.P_rt + (i64)(P.E / c.ep) * cdiv64(P.P_e, etp);
        buf = min((i64)2, copies * Ls) * (i64)P.wb * p_layer;
    }
    const i64 a_tok = c.rec == PF_REC_NONE ? P.a_full : (c.rec == PF_REC_SELECTIVE ? P.a_sel : P.a_ckpt);
    const i64 a_layer = cdiv64(t * a_tok, tp);
    // activation bytes of one microbatch across the rank's Ls layers (leading dense layers hold less)
    i64 a_rank = (Ls - nd0) * a_layer;
    if (nd0) {
        const i64 a_tok_d = c.rec == PF_REC_NONE ? P.a_full_d : (c.rec == PF_REC_SELECTIVE ? P.a_sel_d : P.a_ckpt);
        a_rank += nd0 * cdiv64(t * a_tok_d, tp);
    }
    i64 act;
    if (D.kind == PF_KIND_1F1B)
        act = min(pp, m) * a_rank;
    else if (D.kind == PF_KIND_INTERLEAVED)   // chunks in flight, each a v-th of the rank's layers
        act = min(pp * D.v_eff + pp - 1, m * D.v_eff) * a_rank / (i64)D.v_eff;
    else
        act = min(pp + 1, m) * a_rank;
    if (c.rec == PF_REC_FULL) act += cdiv64(t * P.a_full, tp);
    if (owns_head && P.count_embeddings) act += 4 * cdiv64(t * (i64)P.vocab, tp);
    M.mem = (i64)(P.wb + P.gb) * n_all + M.bytes_o + buf + act + P.reserved_bytes;
}

// Per-layer and per-step time terms shared by the analytic scorer and the simulator.
struct TrainTimes {
    float F_l, B_l, headF, p, T_dp, T_opt;
    float F_ld, B_ld;   // a leading dense layer (0 when the model has none)
    float cD, cE, rc, tpc, a2a;   // a MoE layer's parts: dense and expert compute, recompute, TP and EP collectives
};

template <typename RI>
__device__ __forceinline__ void train_times(const DevPlan &P, const TrainTuple &c, const TrainDerived<RI> &D,
                                            const TrainMem &M, TrainTimes &T)
{
    const DevKern &kn = P.kern[c.kv];
    const float t = (float)D.t, tp = (float)c.tp;
    const float dense_rate = tp * P.peak_flops * P.eff_dense;
    const float cD = fdiv(t * P.f_dense, dense_rate);
    const float cE = fdiv(t * P.f_exp, tp * P.peak_flops * kn.dtype_mult * kn.eff[D.bucket]);
    const float cF = cD + cE, cB = P.bwd_factor * cF;
    float rc = 0.f;
    if (c.rec == PF_REC_SELECTIVE)
        rc = (2.f / 3.f) * (cE + fdiv(t * P.f_sh, dense_rate));
    else if (c.rec == PF_REC_FULL)
        rc = cF;
    const i64 act_bytes = (i64)P.ab * (i64)D.t * (i64)P.H;  // one activation tensor of the microbatch
    const float tpc = 2.f * t_allreduce(c.tp, (float)act_bytes, link_of(P, c.tp));
    const float a2a = 2.f * t_alltoall(c.ep, fdiv((float)(act_bytes * P.K), tp), link_of(P, (i64)c.tp * c.ep));
    // the hiding benefit is conditioned out when the optimizer is offloaded (Sec. 5 RQ2)
    const float hid = (D.ov && c.sh != PF_SHARD_ZERO1_OFFLOAD) ? P.sched[c.s].hide_frac * a2a : 0.f;
    const float xF = a2a - fminf(hid, cF);
    const float xB = a2a - fminf(hid, cB + rc);
    T.cD = cD; T.cE = cE; T.rc = rc; T.tpc = tpc; T.a2a = a2a;
    T.F_l = cF + tpc + xF;
    T.B_l = cB + rc + tpc + xB + (c.rec == PF_REC_FULL ? tpc + xF : 0.f);
    T.headF = fdiv(t * P.f_head, dense_rate);
    // a leading dense layer: no experts, no all-to-all
    T.F_ld = T.B_ld = 0.f;
    if (P.L_dense > 0) {
        const float cDd = fdiv(t * P.f_dense_d, dense_rate);
        const float rcd = c.rec == PF_REC_NONE ? 0.f
                          : (c.rec == PF_REC_SELECTIVE ? (2.f / 3.f) * fdiv(t * P.f_mlp_d, dense_rate) : cDd);
        T.F_ld = cDd + tpc;
        T.B_ld = P.bwd_factor * cDd + rcd + tpc + (c.rec == PF_REC_FULL ? tpc : 0.f);
    }
    T.p = 0.f;
    if (c.pp > 1) {
        Link lw = link_of(P, (i64)D.world);
        T.p = fdiv((float)act_bytes, tp * lw.bw) + lw.alpha;
    }
    Link ldp = link_of(P, (i64)c.tp * (i64)D.dp);
    const float gw = (float)(P.gb + P.wb);
    T.T_dp = t_allreduce((i64)D.dp, gw * (float)M.N_dense, ldp) + t_allreduce((i64)D.edp, gw * (float)M.N_exp, ldp);
    T.T_opt = fdiv(2.f * (float)M.bytes_o, P.hbm_bw);
    if (c.sh == PF_SHARD_ZERO1_OFFLOAD) {
        // the step runs on the host: the shard's gradients go down, its updated weights come back
        T.T_opt = fdiv(gw * (float)M.n_shard, P.bw_host);
    } else if (c.sh == PF_SHARD_FSDP) {
        // per microbatch: parameters gathered for forward and again for backward, gradients reduce-scattered
        const float ag = t_allgather((i64)D.dp, (float)P.wb * (float)M.N_dense, ldp) +
                         t_allgather((i64)D.edp, (float)P.wb * (float)M.N_exp, ldp);
        const float rs = t_allgather((i64)D.dp, (float)P.gb * (float)M.N_dense, ldp) +
                         t_allgather((i64)D.edp, (float)P.gb * (float)M.N_exp, ldp);
        T.T_dp = (float)D.m * (2.f * ag + rs);
    }
}

// Makespan of one MoE layer pass on two streams (Sec. 3.2: the simulator models the overlap of compute and
// communication explicitly).  Compute stream: the dense part A, then n expert chunks; communication stream: n
// dispatch chunks (ready once A is done), then the combine chunks as their expert chunks finish -- the order a
// first-ready-first-served stream produces, since every dispatch is ready before any combine.
__device__ __forceinline__ float two_stream_layer(float A, float e_tot, float d_tot, float c_tot, int n)
{
    const float inv = fdiv(1.f, (float)n);
    const float e = e_tot * inv, d = d_tot * inv, c = c_tot * inv;
    float comm = A;
    for (int i = 0; i < n; i++) comm += d;          // the stream is busy with dispatches until here
    float dend = A, eend = A;
    for (int i = 0; i < n; i++) {
        dend += d;
        eend = fmaxf(eend, dend) + e;               // expert chunk i: after chunk i-1 and its dispatch
        comm = fmaxf(comm, eend) + c;               // combine chunk i
    }
    return comm;
}

// tokens/s/GPU from a pipeline time, with the realization taxes of the plans that pay them
template <typename RI>
__device__ __forceinline__ float train_price(const DevPlan &P, const TrainTuple &c, const TrainDerived<RI> &D,
                                             const TrainTimes &T, float T_pipe)
{
    const float T_step = T_pipe + (1.f - P.dp_overlap_frac) * T.T_dp + T.T_opt + P.step_overhead;
    float tput = fdiv((float)(P.gbs * (i64)P.seq), T_step * (float)D.world);
    const DevKern &kn = P.kern[c.kv];
    if (!kn.is_native) tput = fdiv(tput, 1.f + kn.patch_ovh);
    if (D.ov) tput = fdiv(tput, 1.f + P.sched[c.s].sched_ovh);
    // the contention penalty prices exactly the offloaded-and-overlapped plans (Sec. 3.2)
    if (D.ov && c.sh == PF_SHARD_ZERO1_OFFLOAD) tput = fdiv(tput, 1.f + P.offload_overlap_penalty);
    return tput;
}

// closed-form pipeline time per schedule class
template <typename RI>
__device__ __forceinline__ float train_pipe_analytic(const DevPlan &P, const TrainTuple &c, const TrainDerived<RI> &D,
                                                     const TrainTimes &T)
{
    const float pp = (float)c.pp, m = (float)D.m;
    // the slower of the two extreme ranks: the first (most leading dense layers) and the last (fewest)
    float Fr = (float)D.Ls * T.F_l, Br = (float)D.Ls * T.B_l;
    if (P.L_dense > 0) {
        const float F0 = (float)(D.Ls - D.nd0) * T.F_l + (float)D.nd0 * T.F_ld;
        const float B0 = (float)(D.Ls - D.nd0) * T.B_l + (float)D.nd0 * T.B_ld;
        const float F1 = (float)(D.Ls - D.nd_last) * T.F_l + (float)D.nd_last * T.F_ld;
        const float B1 = (float)(D.Ls - D.nd_last) * T.B_l + (float)D.nd_last * T.B_ld;
        const bool first_slower = F0 + B0 > F1 + B1;
        Fr = first_slower ? F0 : F1;
        Br = first_slower ? B0 : B1;
    }
    const float F = Fr + fdiv(T.headF, pp);
    const float B = Br + P.bwd_factor * fdiv(T.headF, pp);
    if (D.kind == PF_KIND_1F1B) return (m + pp - 1.f) * (F + B) + 2.f * (pp - 1.f) * T.p;
    if (D.kind == PF_KIND_INTERLEAVED)
        return (m + fdiv(pp - 1.f, (float)D.v_eff)) * (F + B) + 2.f * (float)(D.Q - 1) * T.p;
    return m * (F + B) + fmaxf(pp - 2.f, 0.f) * B + fdiv(F + B, P.dualpipe_startup_div) + 2.f * (pp - 1.f) * T.p;
}

// ------------------------------------------------------------------ serving

struct ServeTuple {
    int kv, chunk, batch, dpa, ep, tp, scen;
};

// Rules 1-4 for a serving layout.  first_rule as for training.
template <typename RI>
__device__ __forceinline__ int serve_layout_rules(const DevPlan &P, const ServeTuple &c, int first_rule,
                                                  bool have_batch)
{
    RI world = (RI)P.world, tp = (RI)c.tp, ep = (RI)c.ep;
    if (first_rule <= 1) {
        if (world % tp != 0) return PF_R_WORLD;
        if (c.dpa) {
            // dp-attention: the data-parallel width world/tp must equal ep (Sec. 2.1, boundary B5)
            if (world / tp != ep || c.ep < 2) return PF_R_WORLD;
        } else {
            // experts shard inside the tensor-parallel world: ep * moe_dp == tp (Sec. 4)
            if (tp % ep != 0) return PF_R_WORLD;
        }
    }
    if (first_rule <= 2) {
        if (c.tp > P.G || P.nh % c.tp != 0) return PF_R_TP;
    }
    if (first_rule <= 3) {
        int moe_tp = c.dpa ? c.tp : c.tp / c.ep;
        if (P.E % c.ep != 0 || P.F % moe_tp != 0) return PF_R_EP;
    }
    if (first_rule <= 4 && have_batch) {
        if (c.dpa && c.batch % c.ep != 0) return PF_R_BATCH;
    }
    return 0;
}

struct ServeOut {
    int reason;
    float tput;
    i64 mem;
    i64 m_e = 0;       // decode-step tokens per expert and its bucket (set once rule 8 is reached)
    int bucket = 0;
    uint32_t why = 0;  // PF_WHY_* bits of a feasible plan
};

template <typename RI>
__device__ __forceinline__ void serve_eval(const DevPlan &P, const ServeTuple &c, int first_rule, int Pn, int On,
                                           ServeOut &out)
{
    out.tput = 0.f;
    out.mem = 0;
    int r = serve_layout_rules<RI>(P, c, first_rule, true);
    if (r) {
        out.reason = r;
        return;
    }
    const int n_eng = c.dpa ? c.tp * c.ep : c.tp;
    const int moe_tp = n_eng / c.ep;
    const int b_loc = c.dpa ? c.batch / c.ep : c.batch;
    const RI m_e = ((RI)c.batch * (RI)P.K) / (RI)P.E;
    const RI m_ep = ((RI)c.chunk * (RI)P.K) / (RI)P.E;
    const int b = me_bucket<RI>(m_e), b_pre = me_bucket<RI>(m_ep);
    out.m_e = (i64)m_e;
    out.bucket = b;
    const DevKern &kn = P.kern[c.kv];
    if ((kn.needs_caps & ~P.caps) != 0u || ((kn.avail_mask >> b) & 1u) == 0u || ((kn.avail_mask >> b_pre) & 1u) == 0u) {
        out.reason = PF_R_KERNEL_MISSING;
        return;
    }
    // memory: weights + KV cache + prefill workspace
    const i64 tp = c.tp;
    // leading dense layers carry attention + a plain FFN sharded by tp: no router, no experts
    const i64 Ld = P.L_dense, Lm = P.L - P.L_dense;
    i64 w = Lm * (cdiv64(P.P_dl, tp) * P.wb + P.P_rt * P.wb + (i64)(P.E / c.ep) * cdiv64(P.P_e, moe_tp) * kn.wbytes) +
            2 * cdiv64((i64)P.vocab * P.H, tp) * P.wb;
    if (Ld > 0) w += Ld * cdiv64(P.P_dld, tp) * P.wb;
    const i64 kv_tok = P.attn_kind ? (i64)(P.kv_latent + P.rope_dim) * P.ab : cdiv64(2ll * P.nkv * P.hd, tp) * P.ab;
    const i64 kvc = (i64)b_loc * (i64)(Pn + On) * P.L * kv_tok;
    const i64 act = 8ll * P.ab * c.chunk * P.H;
    out.mem = w + kvc + act + P.reserved_bytes;
    if (out.mem > P.budget_bytes) {
        out.reason = PF_R_MEMORY;
        return;
    }
    // time: per layer max(compute, HBM) + collectives; decode at the mean context length
    const Link lk = link_of(P, n_eng);
    const float peak = P.peak_flops, hbm = P.hbm_bw;
    const float ftp = (float)c.tp, nen = (float)n_eng, bl = (float)b_loc, dk = (float)P.dk, nh = (float)P.nh;
    const float Lf = (float)Lm, Pf = (float)Pn, Of = (float)On;
    const float P_dl = (float)P.P_dl;
    const float dense_rate = ftp * peak * P.eff_dense;
    const float ctx = Pf + Of * 0.5f;
    const float attn_w = fdiv((float)(P.P_dl * P.wb), ftp);
    const float e_loc = (float)(P.E / c.ep);
    const float exp_unit = fdiv((float)(P.P_e * kn.wbytes), (float)moe_tp);
    const float moe_rate = nen * peak * kn.dtype_mult;
    const float KH = (float)((i64)P.K * P.H);
    // decode
    const float touched_d = fminf(e_loc, fmaxf(1.f, fdiv((float)((i64)c.batch * P.K), (float)c.ep)));
    const float t_attn_d = fmaxf(fdiv(bl * (2.f * P_dl + 4.f * ctx * nh * dk), dense_rate), fdiv(attn_w + bl * ctx * (float)kv_tok, hbm));
    const float t_moe_d = fmaxf(fdiv((float)c.batch * P.f_exp, moe_rate * kn.eff[b]), fdiv(touched_d * exp_unit, hbm));
    const float t_com_d = c.dpa ? 2.f * t_alltoall(n_eng, (float)P.ab * bl * KH, lk)
                                : 2.f * t_allreduce(c.tp, (float)((i64)P.ab * c.batch * P.H), lk);
    // a leading dense layer: its weights stream once per step, two all-reduces over tp, no all-to-all
    float t_dl_d = 0.f, t_dl_p = 0.f;
    const float P_dld = (float)P.P_dld, w_dl = fdiv((float)(P.P_dld * P.wb), ftp);
    const Link ltp = link_of(P, c.tp);
    if (Ld > 0)
        t_dl_d = fmaxf(fdiv(bl * (2.f * P_dld + 4.f * ctx * nh * dk), dense_rate), fdiv(w_dl + bl * ctx * (float)kv_tok, hbm)) +
                 2.f * t_allreduce(c.tp, (float)P.ab * bl * (float)P.H, ltp);
    const float T_dec = Lf * (t_attn_d + t_moe_d + t_com_d) + (float)Ld * t_dl_d + P.step_overhead;
    // chunked prefill
    const int nc = (Pn + c.chunk - 1) / c.chunk;
    const float cl = fdiv(Pf, (float)nc);
    const float touched_p = fminf(e_loc, fmaxf(1.f, fdiv(cl * (float)P.K, (float)c.ep)));
    const float t_attn_p = fmaxf(fdiv(cl * (2.f * P_dl + 4.f * (Pf * 0.5f) * nh * dk), dense_rate), fdiv(attn_w, hbm));
    const float t_moe_p = fmaxf(fdiv(cl * P.f_exp, moe_rate * kn.eff[b_pre]), fdiv(touched_p * exp_unit, hbm));
    const float t_com_p = c.dpa ? 2.f * t_alltoall(n_eng, (float)P.ab * cl * KH, lk)
                                : 2.f * t_allreduce(c.tp, (float)P.ab * cl * (float)P.H, lk);
    if (Ld > 0)
        t_dl_p = fmaxf(fdiv(cl * (2.f * P_dld + 4.f * (Pf * 0.5f) * nh * dk), dense_rate), fdiv(w_dl, hbm)) +
                 2.f * t_allreduce(c.tp, (float)P.ab * cl * (float)P.H, ltp);
    const float T_pre = (float)nc * (Lf * (t_attn_p + t_moe_p + t_com_p) + (float)Ld * t_dl_p);
    float tput = fdiv((float)((i64)c.batch * On), (bl * T_pre + Of * T_dec) * nen);
    if (!kn.is_native) tput = fdiv(tput, 1.f + kn.patch_ovh);
    out.tput = tput;
    out.why = domain_why<RI>(P, kn, m_e);
    out.reason = out.why ? PF_FLAG_EXTRAPOLATED : PF_FEASIBLE;
}

}  // namespace pf
