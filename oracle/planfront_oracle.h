/*
 * planfront_oracle.h -- CPU reference ("oracle") for batched MoE parallel-plan scoring.
 *
 * TEST INFRASTRUCTURE ONLY.  This is the plain, slow, candidate-by-candidate definition of
 * what the scoring path computes: fp64 for every floating quantity, int64 for every byte and
 * token count, a full sort for top-k.  It shares no code with the CUDA library and must never
 * be linked, imported or called from the product path; only the tests, the smoke check and
 * the benchmark's CPU-baseline leg use it.
 *
 * What it follows (paper sections):
 *   - plan tuple and its axes ............ Sec. 3.1 (intermediate representation)
 *   - predicate order: emit dry-run rules first, memory gate second ... Sec. 3.3, Fig. 2
 *   - rule list (unmapped schedule class, layer-count divisibility, overlap preconditions,
 *     serving dp == ep, missing kernels) . Sec. 4 "Emitters", Fig. 2, Sec. 5 RQ1
 *   - memory gate, 0.9 usable fraction, expert-DP optimizer shards ... Sec. 2.1, Sec. 5 RQ1
 *   - analytic (closed-form) scorer and the list-scheduling simulator . Sec. 3.2
 *   - realization tax, throughput / (1 + frac) ........................ Sec. 3.2, Table "tax"
 *   - calibration domain m_range [64, 8192], "extrapolated" flag ...... Sec. 3 (P4), Appendix
 *   - top-k invariant (every returned plan passes the predicate) ...... Sec. 3.3
 * The paper prints no equations; where it is silent the reading taken is stated beside each
 * formula in planfront_oracle.c.
 *
 * Pins (what fixes this file to something other than itself) live in the CPU tests:
 * printed memory numbers (72 GB budget, 21.59 GB expert optimizer state, the 10.8 / 21.59 GB
 * ep8 -> ep4 -> ep2 increments), the tax rule, rule outcomes the paper states (27 layers vs
 * pp*v, serving dp != ep, DualPipe unmapped), the 1F1B bubble closed form, the interleaved
 * closed form, brute-force enumeration of the tiny space, and monotonicity invariants.
 * Later additions and their pins: the operation tally (hand counts); the sharding dimension (zero1
 * bit-identity, the printed optimizer sizes, one-rank special cases, the tax rule); the calibration
 * domain (inclusive range, unattached = factory model); leading dense layers (a reconstructed
 * reference model reproduces the printed 0.892e9 dense parameters and 1.34 / 22.93 GB optimizer
 * state); the two-stream layer timeline (an independent event-driven simulation, closed forms).
 * PARITY UNPINNED: absolute throughputs (the paper's cost constants are not published), the
 * DualPipe analytic closed form and its startup divisor, the serving time model, the absolute
 * times of the offloaded and fully sharded regimes, the activation and time formulas of a leading
 * dense layer beyond its FLOP count, and the choice of the two-stream timeline's op graph (the
 * paper names the ingredients, not the graph).
 */
#ifndef PLANFRONT_ORACLE_H
#define PLANFRONT_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORC_MAX_SCHED 8
#define ORC_MAX_KERN 16
#define ORC_NBUCKET 8
#define ORC_MAX_AXES 11
#define ORC_MAX_RANKS 32   /* simulator domain: pp <= 32 */
#define ORC_MAX_V 8        /* simulator domain: virtual stages per rank <= 8 */
#define ORC_SIM_WINDOW 64  /* simulated microbatches per step at most */

/* reason codes (first failing rule, in this order) */
enum {
    ORC_FEASIBLE = 0,
    ORC_R_WORLD = 1,
    ORC_R_TP = 2,
    ORC_R_EP = 3,
    ORC_R_BATCH = 4,
    ORC_R_VSTAGE = 5,
    ORC_R_LAYERS = 6,
    ORC_R_MICROBATCH = 7,
    ORC_R_KERNEL_MISSING = 8,
    ORC_R_UNMAPPED_SCHEDULE = 9,
    ORC_R_OVERLAP_PRECOND = 10,
    ORC_R_MEMORY = 11,
    ORC_FLAG_EXTRAPOLATED = 0x80
};

enum { ORC_KIND_1F1B = 0, ORC_KIND_INTERLEAVED = 1, ORC_KIND_DUALPIPE = 2 };
enum { ORC_REC_NONE = 0, ORC_REC_SELECTIVE = 1, ORC_REC_FULL = 2 };
/* memory sharding (Sec. 3.1, memory plan): optimizer state sharded / and kept in host memory / parameters and
 * gradients sharded as well */
enum { ORC_SHARD_ZERO1 = 0, ORC_SHARD_ZERO1_OFFLOAD = 1, ORC_SHARD_FSDP = 2 };
enum { ORC_SIM_OK = 0, ORC_SIM_UNSUPPORTED = 1, ORC_SIM_STALL = 2 };

typedef struct {
    int64_t L, H, nh, nkv, hd;
    int64_t attn_kind; /* 0 MHA/GQA, 1 MLA */
    int64_t kv_latent, rope_dim;
    int64_t E, K, F, S, Fs;
    int64_t seq, vocab;
    int64_t wb, gb, ob, ab; /* bytes: weight, gradient, optimizer state per parameter, activation */
    int64_t n_mats;         /* matrices per expert FFN (3 = gate, up, down) */
    int64_t count_embeddings;
    /* DeepSeek-style stacks: the first L_dense layers have a plain FFN of width F_dense instead of experts
     * (0 = every layer is MoE); hd_q: query head dimension where it differs from hd (MLA: nope + rope; 0 = hd) */
    int64_t L_dense, F_dense, hd_q;
} orc_model_t;

typedef struct {
    int64_t G;            /* GPUs per node */
    int64_t budget_bytes; /* usable HBM per GPU (caller: 0.9 x capacity) */
    int64_t reserved_bytes;
    int64_t caps; /* bit 0: fp8, bit 1: device-initiated communication */
    double peak_flops, hbm_bw, bw_intra, bw_inter, alpha_intra, alpha_inter;
    double bw_host; /* host link of one GPU, bytes/s (offloaded optimizer) */
    int64_t gpu_id; /* which GPU model the modeled cluster has (an id the caller assigns) */
} orc_cluster_t;

typedef struct {
    int64_t phase;      /* 0 train, 1 serve */
    int64_t gbs;        /* train: sequences per step */
    int64_t world;      /* serve: the cluster's world size */
    int64_t n_scen;     /* serve: number of (prompt, output) scenarios */
    const int64_t *scen_P;
    const int64_t *scen_O;
} orc_workload_t;

typedef struct {
    double eff_dense, bwd_factor, dp_overlap_frac, dualpipe_startup_div, step_overhead;
    double offload_overlap_penalty; /* realization tax of an offloaded-and-overlapped plan (Sec. 3.2) */
} orc_consts_t;

typedef struct {
    int64_t kind, overlap, mapped;
    double hide_frac, sched_ovh;
    /* what the timeline simulator needs about the overlap (Sec. 3.1 "schedule"): the all-to-all is cut into
     * n_chunks pieces (0: the simulator uses hide_frac like the analytic scorer), and while communication
     * kernels run beside compute they hold sm_frac of the SMs */
    int64_t n_chunks;
    double sm_frac;
} orc_sched_t;

typedef struct {
    int64_t needs_caps, avail_mask, is_native, wbytes;
    double dtype_mult, eff[ORC_NBUCKET], patch_ovh;
    int64_t dtype; /* id of the variant's compute dtype (0 bf16, 1 fp8, ...) for the calibration domain */
} orc_kern_t;

/* Calibration domain of the constants (principle P4, Appendix "Testbeds and calibration domains"): the GPU,
 * the dtypes and the tokens-per-expert range they were fit over.  A query outside it is flagged extrapolated;
 * with no domain attached the check is vacuously true and nothing is flagged. */
typedef struct {
    int64_t attached;
    int64_t gpu_id;     /* -1: any GPU */
    int64_t dtype_mask; /* bit d: dtype id d is covered */
    int64_t m_lo, m_hi; /* tokens per expert, inclusive */
} orc_domain_t;
/* why a candidate is extrapolated (bits) */
enum { ORC_WHY_GPU = 1, ORC_WHY_DTYPE = 2, ORC_WHY_M_LOW = 4, ORC_WHY_M_HIGH = 8 };

typedef struct {
    int64_t ep_scope;   /* 0: ep | dp, 1: ep | dp*tp */
    int64_t layer_mode; /* 0: L mod (pp*v) == 0, 2: balanced uneven split, pp*v <= L */
    int64_t tp_max, world_min, world_max;
    int64_t enforce_realizability;
} orc_rules_t;

/* axis value lists, least-significant digit first.
 * train: kv, rec, sched, mb, v, ep, pp, tp, dp, world [, shard]   (10 or 11 axes; no shard axis = zero1)
 * serve: kv, chunk, batch, dpa, ep, tp, scen             (7 axes) */
typedef struct {
    int64_t n_axes;
    int64_t len[ORC_MAX_AXES];
    const int64_t *val[ORC_MAX_AXES];
} orc_axes_t;

typedef struct {
    orc_model_t model;
    orc_cluster_t cluster;
    orc_workload_t workload;
    orc_consts_t consts;
    int64_t n_sched;
    orc_sched_t sched[ORC_MAX_SCHED];
    int64_t n_kern;
    orc_kern_t kern[ORC_MAX_KERN];
    orc_rules_t rules;
    orc_axes_t axes;
    orc_domain_t domain;
} orc_problem_t;

/* candidate-independent model constants (exact integers) */
typedef struct {
    int64_t dk, P_attn, P_rt, P_e, P_sh, P_dl, P_emb;
    int64_t a_attn, a_fix, a_ffn, a_full, a_sel, a_ckpt;
    int64_t f_attn, f_rt, f_sh, f_dense, f_exp, f_head;
    /* a leading dense layer: parameters that shard by tp, activation bytes per token, forward FLOPs per token */
    int64_t P_dld, a_full_d, a_sel_d, f_mlp_d, f_dense_d;
} orc_derived_t;

/* everything computed for one candidate; unfilled parts stay 0 */
typedef struct {
    /* decoded tuple (train names; serve: chunk->mb slot unused, see fields below) */
    int64_t kv, rec, sched, mb, v, ep, pp, tp, dp, world, shard;
    int64_t chunk, batch, dpa, scen; /* serve */
    /* derived integers */
    int64_t kind, ov, v_eff, m, t, Q, Lc, Ls, edp, m_e, bucket, bucket_pre;
    int64_t nd0, nd_last; /* leading dense layers on the first and on the last rank */
    /* memory terms */
    int64_t N_dense, N_exp, bytes_w, bytes_g, bytes_o_dense, bytes_o_expert, bytes_o, bytes_a, bytes_buf, mem;
    /* time terms */
    double cF, cB, rc, tpc, a2a, xF, xB, F_l, B_l, headF, F, B, p, T_pipe, T_dp, T_opt, T_step;
    double T_dec, T_pre; /* serve */
    double F_ld, B_ld;   /* a leading dense layer's forward and backward time */
    double cD, cE;       /* per-layer forward compute: dense part (attention, router, shared experts), experts */
    double tput_unpriced, tput;
    int64_t reason;
    int64_t why; /* ORC_WHY_* bits behind the extrapolated flag (feasible candidates only) */
} orc_detail_t;

int64_t orc_budget_bytes(int64_t hbm_bytes); /* floor(0.9 * capacity), in integers */
void orc_derive(const orc_model_t *m, orc_derived_t *d);
uint64_t orc_space_size(const orc_problem_t *pb);

/* Operation tally for the ALU roofline.  Only a build with -DORACLE_COUNT_OPS counts; the plain build
 * returns zeros.  out[0] integer ops, out[1] floating ops, out[2] candidates, since the last reset. */
int orc_ops_enabled(void);
void orc_ops_reset(void);
void orc_ops_read(int64_t out[3]);

/* Makespan of one MoE layer pass on two streams (Sec. 3.2: the simulator models the overlap of compute and
 * communication explicitly).  Compute stream: the dense part A, then n expert chunks of e_tot / n; communication
 * stream: n dispatch chunks of d_tot / n (ready once A is done) and n combine chunks of c_tot / n (chunk i ready
 * once expert chunk i is done); expert chunk i needs dispatch chunk i.  Each stream runs the ready op that became
 * ready first (ties: lower op number; dispatches are numbered before combines). */
double orc_two_stream_layer(double A, double e_tot, double d_tot, double c_tot, int n);

/* score one candidate: fills detail (may be NULL); returns the reason byte */
int orc_eval(const orc_problem_t *pb, uint64_t idx, orc_detail_t *detail);

/* score [first, first+count); any output may be NULL; uses OpenMP threads when n_threads > 1.
 * returns the number of threads actually used */
int orc_score_range(const orc_problem_t *pb, uint64_t first, uint64_t count, uint8_t *reason,
                    double *tput, int64_t *mem, int n_threads);

/* top-k among entries with (reason & 0x7f) == 0, by (tput desc, idx asc): full sort.
 * idx[i] = first + i for the dense arrays given.  returns the number written (<= k) */
uint64_t orc_topk(const uint8_t *reason, const double *tput, uint64_t first, uint64_t count,
                  uint64_t k, uint64_t *out_idx, double *out_score);
/* same, over an explicit index list (re-ranking of survivors) */
uint64_t orc_topk_list(const uint64_t *idx, const double *score, uint64_t n, uint64_t k,
                       uint64_t *out_idx, double *out_score);

/* survivors: the s_max best feasible candidates inside the simulator domain, sorted by idx */
uint64_t orc_select_survivors(const orc_problem_t *pb, const uint8_t *reason, const double *tput,
                              uint64_t first, uint64_t count, uint64_t s_max, uint64_t *out_idx);

/* --- serving: one score per plan over the whole length mix (Sec. 5 RQ3 ranks serving PLANS) ---
 * The serving space lists every plan once per (prompt, output) scenario; the scenario axis is the most
 * significant one, so candidate idx = plan + n_plans * scenario_digit.  A plan is feasible iff it is feasible
 * in every scenario (its reason is that of the first failing scenario); its score is total output tokens over
 * total time, which for per-scenario throughputs tput_i and output lengths O_i is the O-weighted harmonic mean
 * sum(O_i) / sum(O_i / tput_i).  Bit 7 (extrapolated) is the OR over scenarios. */
uint64_t orc_serve_plan_count(const orc_problem_t *pb);
void orc_aggregate_serving(const orc_problem_t *pb, const uint8_t *reason, const double *tput,
                           uint8_t *plan_reason, double *plan_tput);

/* --- simulator tier --- */
/* op encoding for per-rank orders: bit 0 = backward, bit 1 = direction (DualPipe), bits 2..9 =
 * virtual stage / position q, bits 10.. = microbatch j */
#define ORC_OP(q, j, dir, isb) ((int32_t)(((j) << 10) | ((q) << 2) | ((dir) << 1) | (isb)))
#define ORC_OP_ISB(o) ((o) & 1)
#define ORC_OP_DIR(o) (((o) >> 1) & 1)
#define ORC_OP_Q(o) (((o) >> 2) & 255)
#define ORC_OP_J(o) ((o) >> 10)

/* per-rank static order; out[rank*stride .. ] receives n_ops ops; returns ops per rank, <0 on error
 * kind 0: 1F1B (v ignored), 1: interleaved (m % pp == 0), 2: DualPipe-style (pp == 1 or even, m even) */
int orc_schedule_order(int kind, int pp, int v, int m, int32_t *out, int stride);

/* evaluate a fixed order with per-stage durations; returns makespan, <0 on stall.
 * Fq/Bq have Q entries (Q = pp*v; DualPipe: pp).  p = cross-rank latency */
double orc_makespan(int kind, int pp, int v, int m, const double *Fq, const double *Bq, double p);

uint32_t orc_mix32(uint32_t x);
double orc_jitter(uint32_t seed, uint64_t idx, int q, int is_backward);

/* simulate one survivor; returns status; *tput_sim receives the priced simulated throughput */
int orc_simulate(const orc_problem_t *pb, uint64_t idx, uint32_t seed, double *tput_sim,
                 double *T_pipe_sim);
int orc_simulate_list(const orc_problem_t *pb, const uint64_t *idx, uint64_t n, uint32_t seed,
                      double *tput_sim, uint8_t *status, int n_threads);

#ifdef __cplusplus
}
#endif
#endif
