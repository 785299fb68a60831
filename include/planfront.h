/*
 * planfront.h -- C ABI of the B200 plan-scoring library (libplanfront.so).
 *
 * The library scores every candidate of a mixed-radix plan space on one GPU:
 *   (model spec, modeled-cluster spec, plan-axis ranges, kernel/overhead tables)
 *     -> (feasibility reason, predicted tokens/s/GPU, peak memory per GPU, top-k plan indices),
 * then re-ranks the best survivors with a per-candidate pipeline-schedule simulation.
 * This is the search loop of the paper's three-tier optimizer (Sec. 3.3) with its realizability
 * predicate (Sec. 3.3, Fig. 2), dual-fidelity cost model (Sec. 3.2) and realization tax (Sec. 3.2),
 * evaluated for all candidates at once instead of one Python call per plan.
 *
 * Conventions
 *   - plain C, no exceptions; every call returns an int32 status (PF_OK = 0, negative = error).
 *   - "d_" pointers are DEVICE pointers owned by the caller; everything else is HOST memory.
 *   - the library allocates no output or workspace memory: the caller passes raw pointers and sizes.
 *     (pf_plan_create takes one block of device memory for the plan's tables -- tens of KB; 5 bytes per block of
 *     candidates for the visiting order -- two streams and six events; pf_plan_destroy waits for the device and
 *     hands them to a small per-device cache for the next plan instead of releasing them.)
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All device work is
 *     enqueued on it and the calls do not synchronize; results are valid once the stream has been
 *     synchronized by the caller.  pf_search_host is the exception: it takes host buffers and returns
 *     after its copies have completed.
 *   - spec structs are copied by pf_plan_create; the caller may free them afterwards.
 *   - a handle may be used from one thread at a time, on the device that was current at create: every call
 *     that enqueues device work returns PF_EINVAL (nothing launched) when another device is current.
 *     Different handles may be used from different threads at the same time (what they share -- the caches above,
 *     the kernels' shared-memory limits -- is locked).
 *   - candidates are addressed by a linear index: idx = sum_a digit_a * prod_{b<a} len_b, axes listed
 *     least-significant first.  train axes: kv, rec, sched, mb, v, ep, pp, tp, dp, world [, shard];
 *     serve axes: kv, chunk, batch, dpa, ep, tp, scen.  An axis value list {0} for dp / world / v means
 *     "derived" (dp = world/(tp*pp); world = tp*pp*dp; v = 2 for interleaved schedules, else 1).
 */
#ifndef PLANFRONT_H
#define PLANFRONT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PF_VERSION 100
#define PF_MAX_AXES 11
#define PF_MAX_AXIS_LEN 4096
#define PF_MAX_SCHED 8
#define PF_MAX_KERN 16
#define PF_NBUCKET 8
#define PF_K_MAX 1024         /* largest top-k */
#define PF_MAX_SCEN 4096
#define PF_SIM_MAX_RANKS 32   /* simulator domain: pp <= 32 (one lane per pipeline rank) */
#define PF_SIM_MAX_V 8        /* simulator domain: virtual stages per rank <= 8 */
#define PF_SIM_WINDOW 64      /* simulated microbatches per step at most */
#define PF_MAX_COUNT (1ull << 32) /* pf_score / pf_select_survivors take count < PF_MAX_COUNT per call */

/* status codes */
enum {
    PF_OK = 0,
    PF_EINVAL = -1,       /* NULL required pointer, inconsistent spec, k out of range */
    PF_ERANGE = -2,       /* axis length 0 or too long, space size >= 2^63, range outside the space */
    PF_EWORKSPACE = -3,   /* workspace too small or misaligned (needs 256-byte alignment) */
    PF_ECUDA = -4,        /* a CUDA runtime call failed; see pf_last_cuda_error() */
    PF_EUNSUPPORTED = -5  /* the call does not apply to this plan's phase */
};

/* per-candidate reason byte: 0 = feasible, else the FIRST failing rule in this order (the predicate's
 * fixed order: structural checks, emit dry-run rules, memory gate last -- Sec. 3.3, Fig. 2).
 * Bit 7 is OR-ed into a feasible candidate whose tokens-per-expert lies outside the calibration
 * domain [64, 8192] ("extrapolated", Sec. 3 principle P4). */
enum {
    PF_FEASIBLE = 0,
    PF_R_WORLD = 1,
    PF_R_TP = 2,
    PF_R_EP = 3,
    PF_R_BATCH = 4,
    PF_R_VSTAGE = 5,
    PF_R_LAYERS = 6,
    PF_R_MICROBATCH = 7,
    PF_R_KERNEL_MISSING = 8,
    PF_R_UNMAPPED_SCHEDULE = 9,
    PF_R_OVERLAP_PRECOND = 10,
    PF_R_MEMORY = 11,
    PF_FLAG_EXTRAPOLATED = 0x80
};

enum { PF_KIND_1F1B = 0, PF_KIND_INTERLEAVED = 1, PF_KIND_DUALPIPE = 2 };
enum { PF_REC_NONE = 0, PF_REC_SELECTIVE = 1, PF_REC_FULL = 2 };
/* memory sharding (Sec. 3.1, memory plan): optimizer state sharded over the data-parallel groups; the same with
 * the state kept in host memory; parameters and gradients sharded as well (with an all-gather working buffer) */
enum { PF_SHARD_ZERO1 = 0, PF_SHARD_ZERO1_OFFLOAD = 1, PF_SHARD_FSDP = 2 };
enum { PF_PHASE_TRAIN = 0, PF_PHASE_SERVE = 1 };
enum { PF_CAP_FP8 = 1, PF_CAP_DEVICE_COMM = 2 };
/* per-survivor simulator status */
enum { PF_SIM_OK = 0, PF_SIM_UNSUPPORTED = 1, PF_SIM_STALL = 2 };

typedef struct {
    int32_t L, H, nh, nkv, hd;
    int32_t attn_kind;            /* 0 MHA/GQA, 1 MLA (compressed KV) */
    int32_t kv_latent, rope_dim;  /* MLA only */
    int32_t E, K, F, S, Fs;       /* routed experts, top-k, expert FFN, shared experts, shared FFN */
    int32_t seq, vocab;
    int32_t wb, gb, ob, ab;       /* bytes per weight / gradient / optimizer state per param / activation */
    int32_t n_mats;               /* matrices per expert FFN (3 = gate, up, down) */
    int32_t count_embeddings;     /* 0/1: embedding + head counted in memory */
    /* DeepSeek-style stacks (0 = not used): the first L_dense layers carry a plain FFN of width F_dense instead
     * of experts; hd_q: query head dimension where it differs from hd (latent attention: nope + rope dims) */
    int32_t L_dense, F_dense, hd_q;
} pf_model_t;

typedef struct {
    int32_t G;                    /* GPUs per node */
    uint32_t caps;                /* PF_CAP_* bits the modeled cluster has */
    int64_t budget_bytes;         /* usable HBM per GPU: the memory gate rejects mem > budget (Sec. 5 RQ1) */
    int64_t reserved_bytes;       /* added to every candidate's memory */
    float peak_flops, hbm_bw, bw_intra, bw_inter, alpha_intra, alpha_inter;
    float bw_host;                /* host link of one GPU, bytes/s: carries an offloaded optimizer step */
    int32_t gpu_id;               /* which GPU model the cluster has (an id the caller assigns; see pf_domain_t) */
} pf_cluster_t;

typedef struct {
    int32_t phase;                /* PF_PHASE_* */
    int32_t n_scen;               /* serve: number of (prompt, output) length scenarios */
    int64_t gbs;                  /* train: sequences per step */
    int64_t world;                /* serve: world size of the modeled cluster */
    const int32_t *scen_P;        /* host, n_scen entries */
    const int32_t *scen_O;
} pf_workload_t;

typedef struct {
    int32_t n_axes;               /* 10 or 11 (train: 11 with the sharding axis last) or 7 (serve) */
    int32_t len[PF_MAX_AXES];     /* 1 .. PF_MAX_AXIS_LEN */
    const int32_t *val[PF_MAX_AXES]; /* host value lists */
} pf_axes_t;

typedef struct {
    int32_t kind;                 /* PF_KIND_* */
    int32_t overlap;              /* expert all-to-all overlapped with compute */
    int32_t mapped;               /* 0: the toolchain cannot emit this class (Sec. 2.1) */
    float hide_frac;              /* hidden fraction of the all-to-all when overlapped (alpha-table) */
    float sched_ovh;              /* realization overhead, applied as tput / (1 + ovh) when overlap = 1 */
    /* What the timeline simulator needs about the overlap (Sec. 3.1, schedule): the all-to-all is cut into
     * n_chunks pieces, 0..16 (0: pf_simulate uses hide_frac like the analytic scorer; >= 1: it runs the layer's
     * two-stream timeline, Sec. 3.2), and communication kernels hold sm_frac of the SMs, 0 <= sm_frac <= 0.9,
     * while they run beside compute.  pf_score ignores both. */
    int32_t n_chunks;
    float sm_frac;
} pf_sched_t;

typedef struct {
    uint32_t needs_caps;          /* PF_CAP_* bits the variant needs */
    uint32_t avail_mask;          /* bit b: the autotune report has an entry for tokens-per-expert bucket b */
    int32_t is_native;            /* 1: the engine's own kernel, pays no patch overhead */
    int32_t wbytes;               /* expert weight bytes per parameter in serving (2 bf16, 1 fp8) */
    float dtype_mult;             /* peak multiplier of the variant's dtype (1 bf16, 2 fp8) */
    float eff[PF_NBUCKET];        /* efficiency per bucket: m_e <128, 128.., 256.., ... , >=8192 */
    float patch_ovh;              /* realization tax, applied as tput / (1 + ovh) when !is_native */
    int32_t dtype;                /* id of the variant's compute dtype, 0..31 (0 bf16, 1 fp8, ...; see pf_domain_t) */
} pf_kern_t;

/* Calibration domain of the constants (principle P4; Appendix "Testbeds and calibration domains"): the GPU, the
 * dtypes and the tokens-per-expert range they were fit over.  A feasible plan outside it gets PF_FLAG_EXTRAPOLATED;
 * its score is not changed.  With no domain attached nothing is flagged. */
typedef struct {
    int32_t attached;             /* 0: no domain (the factory model) */
    int32_t gpu_id;               /* -1: any GPU */
    uint32_t dtype_mask;          /* bit d: dtype id d is covered */
    int32_t m_lo, m_hi;           /* tokens per expert, inclusive (the paper's domains: [64, 8192]) */
} pf_domain_t;
/* why a plan is extrapolated (bits of pf_report_t.why) */
enum { PF_WHY_GPU = 1, PF_WHY_DTYPE = 2, PF_WHY_M_LOW = 4, PF_WHY_M_HIGH = 8 };

typedef struct {
    float eff_dense, bwd_factor, dp_overlap_frac, dualpipe_startup_div, step_overhead;
    float offload_overlap_penalty; /* realization tax of offloaded-and-overlapped plans, tput / (1 + frac) (Sec. 3.2) */
    int32_t n_sched;
    pf_sched_t sched[PF_MAX_SCHED];
    int32_t n_kern;
    pf_kern_t kern[PF_MAX_KERN];
    pf_domain_t domain;
} pf_tables_t;

typedef struct {
    int32_t ep_scope;             /* 0: ep | dp (EP inside DP, Sec. 4), 1: ep | dp*tp */
    int32_t layer_mode;           /* 0: L mod (pp*v) == 0 (Fig. 2), 2: balanced uneven split, pp*v <= L */
    int32_t tp_max;
    int32_t world_min, world_max;
    int32_t enforce_realizability; /* 0: unconstrained mode, dry-run rules 9-10 skipped (Sec. 3.3) */
} pf_rules_t;

typedef struct {
    int32_t kv, rec, sched, mb, v, ep, pp, tp, dp, world; /* train (dp/world as listed, before derivation) */
    int32_t chunk, batch, dpa, scen;                      /* serve */
    int32_t shard;                                        /* train: PF_SHARD_* (zero1 when the axis is absent) */
} pf_tuple_t;

typedef struct pf_plan pf_plan_t;

int pf_version(void);
const char *pf_strerror(int status);
const char *pf_reason_str(uint8_t reason);
/* text of the last CUDA error seen by this thread's library calls ("" if none) */
const char *pf_last_cuda_error(void);

/* Build a plan space (Sec. 3.1: one normalized tuple carries every knob; Sec. 3.3: enumeration).
 * Validates the specs, derives the candidate-independent constants (parameter, activation and FLOP
 * counts per layer; radices; schedule-order tables for the simulator) and uploads them.
 * A training space may carry the memory-sharding dimension (Sec. 3.1, memory plan) as an 11th, most significant
 * axis with values PF_SHARD_*; without it every plan is zero1.  Such a space needs cluster->bw_host > 0.
 * Errors: PF_EINVAL (NULL pointer, phase/axis-count mismatch, table index out of range, both dp and
 * world derived, a sharding value outside PF_SHARD_*), PF_ERANGE (axis length, value range, space size),
 * PF_ECUDA. */
int pf_plan_create(const pf_model_t *model, const pf_cluster_t *cluster, const pf_workload_t *workload,
                   const pf_axes_t *axes, const pf_tables_t *tables, const pf_rules_t *rules, pf_plan_t **out);
void pf_plan_destroy(pf_plan_t *plan);
uint64_t pf_plan_size(const pf_plan_t *plan); /* N = product of axis lengths */
/* host helper: linear index -> axis values (no rule is applied).  PF_ERANGE if idx >= N. */
int pf_decode(const pf_plan_t *plan, uint64_t idx, pf_tuple_t *out);

/* Score candidates [first, first+count): decode -> realizability rules -> memory gate -> analytic step
 * time -> priced throughput (Sec. 3.2-3.3), and reduce to the k best feasible ones by (tput descending,
 * index ascending) (Sec. 3.3: every returned plan passes the predicate).
 *   d_reason[count] uint8, d_tput[count] float (tokens/s/GPU, 0 when infeasible), d_mem[count] int64
 *   (bytes; 0 when a rule before the memory gate failed) -- each may be NULL (not written); element i
 *   belongs to candidate first+i.
 *   k = 0 skips the top-k; otherwise 1 <= k <= PF_K_MAX and d_topk_idx[k] (uint64, UINT64_MAX in unused
 *   slots), d_topk_score[k] (float, 0 in unused slots), d_topk_count[1] (uint32) are required.
 *   d_workspace: at least pf_score_workspace(plan, count, k) bytes, 256-byte aligned, contents ignored.
 * count < PF_MAX_COUNT per call; larger spaces are scored in chunks and merged with pf_topk_merge.
 * The plan keeps, in device memory it allocated at creation, the order in which the kernel visits the blocks
 * of candidates of its latest range (evaluated blocks first, spread between constant ones); a call on another
 * range rebuilds it on `stream` with two small launches, a call on the same range reuses it.  Device work of
 * calls on one plan must therefore be ordered (one stream, or events between streams); a table that does not
 * hold the call's range -- e.g. its rebuild was captured into a graph that has not run -- is detected on the
 * device and ignored, at some cost in speed only.
 * Errors: PF_EINVAL, PF_ERANGE, PF_EWORKSPACE, PF_ECUDA (launch failure). */
size_t pf_score_workspace(const pf_plan_t *plan, uint64_t count, uint32_t k);
int pf_score(pf_plan_t *plan, uint64_t first, uint64_t count, uint8_t *d_reason, float *d_tput, int64_t *d_mem,
             uint32_t k, uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count, void *d_workspace,
             size_t workspace_bytes, void *stream);

/* pf_score for callers that must not allocate device memory when they call it.  (The paper has no
 * counterpart: this is a deployment convenience of this library.)
 *
 * Who needs it: code that runs where a device allocation is unavailable or forbidden -- a service whose
 * whole device memory is handed to a pool at start-up, a latency-critical loop in which the implicit device
 * synchronization of an allocation is not acceptable, a plugin that is given buffers by its host application
 * and has no allocator of its own.  Such a caller can usually still provide the inputs and the result
 * buffers, but has nowhere to take pf_score's workspace from.
 *
 * Same arguments and results as pf_score, minus the workspace: the scratch memory (work counters and the
 * blocks' candidate key lists) lives in a fixed array of PF_STATIC_SCRATCH_BYTES inside the library's device
 * image.  Every GPU that loads the library carries that array until the process exits.
 *   - The call allocates nothing and frees nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *   - The FIRST call on each device looks up the array's device address (once per device, with that device
 *     current); make that first call before any stream capture begins.
 *   - All calls on one device share the one array, which keeps the previous call's contents; the call clears
 *     the words that must start at zero.  Two calls whose device work overlaps (different streams, different
 *     threads) race on it: issue them on one stream, or order them yourself.
 *   - A request whose workspace need (pf_score_workspace) exceeds PF_STATIC_SCRATCH_BYTES is refused with
 *     PF_EWORKSPACE before anything is launched; use pf_score with your own workspace for it.
 *   - Only the first call on a device may make the CUDA runtime load the library's device image there (the
 *     image holds the array); no later call changes the device's free memory.
 * Errors: as pf_score; PF_ECUDA also if the address look-up fails; PF_EUNSUPPORTED on a device whose ordinal is
 * 64 or more (the per-device address table is that long). */
#define PF_STATIC_SCRATCH_BYTES (4u << 20)
int pf_score_static(pf_plan_t *plan, uint64_t first, uint64_t count, uint8_t *d_reason, float *d_tput,
                    int64_t *d_mem, uint32_t k, uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count,
                    void *stream);

/* Merge two top-k lists (as written by pf_score / pf_simulate, each sorted, with device counts) into the k
 * best of their union, same ordering rule.  Used to combine chunks or shards of one space.  The output
 * may alias neither input.  Errors: PF_EINVAL (k out of range, NULL). */
int pf_topk_merge(uint32_t k, const uint64_t *d_idx_a, const float *d_score_a, const uint32_t *d_count_a,
                  const uint64_t *d_idx_b, const float *d_score_b, const uint32_t *d_count_b,
                  uint64_t *d_idx_out, float *d_score_out, uint32_t *d_count_out, void *stream);

/* Survivor selection for the schedule tier (Sec. 3.3: the top-ranked layouts are refined with the
 * simulator; here the short list is the s_max best instead of ten): among candidates of
 * [first, first+count) that are feasible ((reason & 0x7f) == 0) and inside the simulator's domain
 * (training plan, pp <= PF_SIM_MAX_RANKS, virtual stages <= PF_SIM_MAX_V), the s_max best by
 * (tput descending, index ascending), written as absolute indices in ASCENDING index order.
 *   d_reason / d_tput: the dense outputs of pf_score for the same range (required).
 *   d_surv_idx[s_max] uint64, d_surv_count[1] uint64 (= min(s_max, eligible)).
 * Errors: PF_EINVAL, PF_ERANGE, PF_EWORKSPACE, PF_EUNSUPPORTED (serving plan), PF_ECUDA. */
size_t pf_select_workspace(const pf_plan_t *plan, uint64_t count, uint64_t s_max);
int pf_select_survivors(pf_plan_t *plan, uint64_t first, uint64_t count, const uint8_t *d_reason,
                        const float *d_tput, uint64_t s_max, uint64_t *d_surv_idx, uint64_t *d_surv_count,
                        void *d_workspace, size_t workspace_bytes, void *stream);

/* The same selection in steps, for one space split over several GPUs (candidates are independent, so a rank scores
 * and selects inside a contiguous slice of the index range; only histograms and counts travel).  With ranks
 * r = 0..G-1 holding slices in ascending index order:
 *   1. every rank: pf_select_hist(..., d_cut = NULL, d_hist): 65,536-bin histogram of the HIGH 16 bits of the fp32
 *      score of its eligible candidates; the caller sums the ranks' histograms (as 64-bit counts);
 *   2. pf_select_cut(sum, level 0, s_max, d_cut): the bin in which the running count from the top reaches s_max
 *      (or take_all when no more than s_max are eligible in all);
 *   3. every rank: pf_select_hist(..., d_cut, d_hist): histogram of the LOW 16 bits inside that bin; summed again;
 *   4. pf_select_cut(sum, level 1, 0, d_cut): the threshold score bits, how many candidates lie above it and how
 *      many of those exactly AT it are still needed (need_eq) -- taken in ascending index order, i.e. rank by rank;
 *   5. every rank: pf_select_write(..., d_cut, eq_before, ...) with eq_before = the number of candidates at the
 *      threshold on lower ranks (each rank's count is entry thr_bits & 0xFFFF of its own step-3 histogram): its
 *      survivors in ascending index order.  The ranks' lists, concatenated in rank order, are what
 *      pf_select_survivors returns for the whole space.  d_surv_idx holds surv_cap entries (a slice yields at most
 *      min(count, s_max)); *d_surv_count is the slice's full count even when it exceeds surv_cap.
 * Every call is self-contained (d_workspace: pf_select_workspace bytes, contents ignored).  d_hist: uint32[65536];
 * the sums passed to pf_select_cut: uint64[65536].  Errors as pf_select_survivors. */
typedef struct {
    uint64_t total;      /* eligible candidates in all */
    uint64_t above_hi;   /* eligible with high score bits above bin_hi */
    uint64_t n_gt;       /* eligible with score bits above the threshold */
    uint64_t need_eq;    /* candidates exactly at the threshold that are taken (smallest indices first) */
    uint64_t target;     /* min(s_max, total) once both levels are done: s_max */
    uint32_t bin_hi, thr_bits;
    int32_t take_all;    /* 1: no more than s_max are eligible: everything is taken, no threshold */
    uint32_t reserved;
} pf_select_cut_t;
int pf_select_hist(pf_plan_t *plan, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
                   const pf_select_cut_t *d_cut, uint32_t *d_hist, void *d_workspace, size_t workspace_bytes,
                   void *stream);
int pf_select_cut(const uint64_t *d_hist, int level, uint64_t s_max, pf_select_cut_t *d_cut, void *stream);
int pf_select_write(pf_plan_t *plan, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
                    const pf_select_cut_t *d_cut, uint64_t eq_before, uint64_t *d_surv_idx, uint64_t surv_cap,
                    uint64_t *d_surv_count, void *d_workspace, size_t workspace_bytes, void *stream);

/* Simulator tier (Sec. 3.2: the list-scheduling timeline is the higher-fidelity scorer used to refine
 * schedules).  For each of the n candidates listed in d_surv_idx (n may also be given on the device:
 * if d_n is not NULL the kernel uses min(n, *d_n)): per-stage forward/backward durations from the
 * analytic terms with an exact balanced layer split, +-10% multiplicative jitter from a counter hash
 * of (jitter_seed, idx, stage, F/B), evaluation of the schedule's fixed per-rank order (1F1B,
 * interleaved, DualPipe-style) with cross-rank latency, steady-state extension beyond PF_SIM_WINDOW
 * microbatches, then the same step terms and pricing as pf_score.
 *   d_tput_sim[n] float, d_sim_status[n] uint8 (PF_SIM_*) -- each may be NULL.
 *   top-k outputs as in pf_score, ranking by (tput_sim descending, index ascending); entries past
 *   min(n, *d_n) are ignored.  An infeasible candidate scores 0 with status PF_SIM_UNSUPPORTED; a
 *   feasible one outside the domain keeps its analytic score with PF_SIM_UNSUPPORTED.
 * Errors: PF_EINVAL, PF_EWORKSPACE, PF_EUNSUPPORTED (serving plan), PF_ECUDA. */
size_t pf_simulate_workspace(const pf_plan_t *plan, uint64_t n, uint32_t k);
int pf_simulate(pf_plan_t *plan, const uint64_t *d_surv_idx, uint64_t n, const uint64_t *d_n,
                uint32_t jitter_seed, float *d_tput_sim, uint8_t *d_sim_status, uint32_t k,
                uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count, void *d_workspace,
                size_t workspace_bytes, void *stream);

/* Serving plans ranked over the whole request-length mix (Sec. 5 RQ3 compares serving PLANS; the scored
 * space lists every plan once per (prompt, output) scenario, scenario being the most significant axis, so
 * candidate = plan + n_plans * scenario_digit and n_plans = N / len(scen axis)).
 * Input: the dense d_reason / d_tput of pf_score over the WHOLE space (first = 0, count = N).
 * Per plan: feasible iff feasible in every scenario, else the reason of the first failing scenario and score
 * 0; score = total output tokens / total time = sum(O_i) / sum(O_i / tput_i) over the scenarios; bit 7
 * (extrapolated) is the OR over scenarios.
 *   d_plan_reason[n_plans] uint8, d_plan_tput[n_plans] float -- each may be NULL;
 *   top-k over plans as in pf_score (k = 0 skips it), indices are plan numbers.
 * Errors: PF_EINVAL, PF_EWORKSPACE, PF_EUNSUPPORTED (training plan), PF_ECUDA. */
uint64_t pf_serve_plan_count(const pf_plan_t *plan);
size_t pf_aggregate_workspace(const pf_plan_t *plan, uint32_t k);
int pf_aggregate_serving(pf_plan_t *plan, const uint8_t *d_reason, const float *d_tput, uint8_t *d_plan_reason,
                         float *d_plan_tput, uint32_t k, uint64_t *d_topk_idx, float *d_topk_score,
                         uint32_t *d_topk_count, void *d_workspace, size_t workspace_bytes, void *stream);

/* Host helper (no GPU): the DualPipe-style per-rank op order the simulator uses for pipeline depth pp
 * (1 or even, <= PF_SIM_MAX_RANKS) and m microbatches (even, 2..PF_SIM_WINDOW).  The order is defined by a
 * nominal list scheduling (forward 1 tick, backward 2 ticks, zero latency; ready op with the smallest
 * (ready time, backward first, microbatch, direction); a forward at position q waits while pp - q
 * microbatches of its direction are in flight on the rank).  The paper names the schedule class only
 * (Sec. 3.1); this order is this library's definition of it.
 * out_ops[pp][2*m]: op = (microbatch << 2) | (direction << 1) | is_backward; direction 0 places position q
 * on rank q, direction 1 on rank pp-1-q; each direction carries m/2 microbatches.
 * Errors: PF_EINVAL (shape outside the domain, NULL). */
int pf_dualpipe_order(int pp, int m, uint8_t *out_ops);

/* Whole search on DEVICE buffers in one call: pf_score over the full space (dense outputs + analytic top-k), then,
 * for training plans with s_max > 0, pf_select_survivors and pf_simulate (top-k_sim of the simulated survivors;
 * their dense simulator outputs are not kept).  Results are what the three calls give one after the other; inside
 * one call the scoring kernel also gathers what the selection's first pass would re-read the dense outputs for,
 * so the selection starts at its second pass.  d_reason, d_tput and the top-k buffers are required, d_mem may be
 * NULL; the survivor and simulator buffers are required when the simulator tier runs (d_surv_idx: s_max entries).
 * d_workspace: pf_search_device_workspace() bytes, 256-byte aligned.  Enqueues on `stream`, does not synchronize.
 * (With a simulator tier, parts of the call run on two more streams that belong to the plan -- the reduction of
 * the analytic top-k on one, the kernel that streams the constant blocks of the dense outputs on the other --
 * forked from and joined back into `stream` by events inside the call: all outputs are complete when the work the
 * call put on `stream` is done, and the call can be captured into a graph.)
 * Errors as the calls above. */
size_t pf_search_device_workspace(const pf_plan_t *plan, uint32_t k, uint64_t s_max, uint32_t k_sim);
int pf_search(pf_plan_t *plan, uint32_t k, uint64_t s_max, uint32_t k_sim, uint32_t jitter_seed, uint8_t *d_reason,
              float *d_tput, int64_t *d_mem, uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count,
              uint64_t *d_surv_idx, uint64_t *d_surv_count, uint64_t *d_sim_topk_idx, float *d_sim_topk_score,
              uint32_t *d_sim_topk_count, void *d_workspace, size_t workspace_bytes, void *stream);

/* Whole search with HOST result buffers (the call a user without device code makes): scores the full
 * space, returns the analytic top-k and -- for training plans with s_max > 0 -- the simulator-refined
 * top-k_sim over the s_max best survivors.  Dense per-candidate outputs are copied back only for the
 * non-NULL h_* pointers (N elements each).  d_workspace must hold pf_search_workspace() bytes of DEVICE
 * memory (it carries the dense arrays, the survivor list and the per-kernel workspaces).
 * Returns after all copies have completed.  Errors as the calls above. */
size_t pf_search_workspace(const pf_plan_t *plan, uint32_t k, uint64_t s_max, uint32_t k_sim);
int pf_search_host(pf_plan_t *plan, uint32_t k, uint64_t s_max, uint32_t k_sim, uint32_t jitter_seed,
                   uint8_t *h_reason, float *h_tput, int64_t *h_mem, uint64_t *h_topk_idx, float *h_topk_score,
                   uint32_t *h_topk_count, uint64_t *h_sim_topk_idx, float *h_sim_topk_score,
                   uint32_t *h_sim_topk_count, uint64_t *h_surv_count, void *d_workspace,
                   size_t workspace_bytes, void *stream);

/* A compact view of dense scoring outputs (the paper's search reports which plans pass and why the others fail,
 * Sec. 3.3: "the pruned set is attributable"; in its spaces, as in this library's, a few candidates in ten thousand
 * pass).  From d_reason / d_tput / d_mem of candidates [first, first+count), as pf_score wrote them:
 *   d_hist[PF_REASON_BINS] uint64: candidates per reason code (entry 0: feasible, flagged ones included);
 *   d_mask (may be NULL): ceil(count / 8) bytes, bit (i mod 8) of byte i / 8 set iff candidate first + i is feasible;
 *   d_records[record_cap] (record_cap may be 0): the feasible candidates in ascending index order -- index,
 *     peak bytes (0 when d_mem is NULL), tokens/s/GPU, reason byte (0 or PF_FLAG_EXTRAPOLATED); when more than
 *     record_cap are feasible the first record_cap are written;
 *   d_n_feasible[1] uint64: how many are feasible (compare with record_cap to detect a truncated list).
 * d_workspace: pf_compact_workspace(count) bytes, 256-byte aligned.  Enqueues on `stream`, does not synchronize.
 * Errors: PF_EINVAL, PF_ERANGE, PF_EWORKSPACE, PF_ECUDA. */
#define PF_REASON_BINS 16
typedef struct {
    uint64_t idx;
    int64_t mem;
    float tput;
    uint8_t reason, pad[3];
} pf_record_t;
size_t pf_compact_workspace(uint64_t count);
int pf_compact(pf_plan_t *plan, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
               const int64_t *d_mem, uint64_t *d_hist, uint8_t *d_mask, pf_record_t *d_records, uint64_t record_cap,
               uint64_t *d_n_feasible, void *d_workspace, size_t workspace_bytes, void *stream);

/* pf_search_host with the compact view in place of the dense per-candidate arrays: what crosses the host link is
 * the reason histogram (h_hist[PF_REASON_BINS]), the feasibility bits (h_mask, N / 8 bytes, may be NULL), the
 * feasible plans' records (h_records[record_cap], may be NULL with record_cap 0) and their number (h_n_feasible),
 * besides the two top-k lists -- on the 1.8e8-candidate space about 23 MB instead of 2.3 GB.
 * d_workspace: pf_search_compact_workspace() bytes of DEVICE memory.  Returns after all copies have completed
 * (the view is taken, and its copies start, as soon as the candidates are scored, beside the selection and the
 * simulator).  Every host pointer may be pageable or page-locked memory.  The small results (histogram, count, top-k
 * lists) pass through a page-locked block of the library's own.  h_mask and h_records are written directly: into
 * page-locked memory beside the search, into pageable memory at its end.  A page-locked h_mask is moreover filled
 * in two parts -- a copy of zeros to the whole of it that starts with the call, and, once the candidates are
 * scored, device writes of the few 2 KB stretches that hold a feasible plan -- so its N / 8 bytes cross the host
 * link beside the search instead of behind it.  Errors as pf_search_host. */
size_t pf_search_compact_workspace(const pf_plan_t *plan, uint32_t k, uint64_t s_max, uint32_t k_sim,
                                   uint64_t record_cap);
int pf_search_host_compact(pf_plan_t *plan, uint32_t k, uint64_t s_max, uint32_t k_sim, uint32_t jitter_seed,
                           uint64_t *h_hist, uint8_t *h_mask, pf_record_t *h_records, uint64_t record_cap,
                           uint64_t *h_n_feasible, uint64_t *h_topk_idx, float *h_topk_score, uint32_t *h_topk_count,
                           uint64_t *h_sim_topk_idx, float *h_sim_topk_score, uint32_t *h_sim_topk_count,
                           uint64_t *h_surv_count, void *d_workspace, size_t workspace_bytes, void *stream);

/* Extrapolation report for a list of plans, e.g. a top-k list (principle P4: a query outside the calibration
 * domain is flagged, not silently trusted).  Entry i of d_out describes plan d_idx[i]: its reason byte as pf_score
 * writes it, the PF_WHY_* bits behind an extrapolated flag, its tokens per expert and efficiency bucket (0 where
 * the plan fails before they are derived).  An index of UINT64_MAX (an unused top-k slot) or >= N gives
 * reason 0xFF.  d_n (device, may be NULL): only the first min(n, *d_n) entries are written.  One small launch on
 * `stream`, no workspace.  Errors: PF_EINVAL (NULL pointer), PF_ECUDA. */
typedef struct {
    uint8_t reason, why;
    uint16_t bucket;
    uint32_t reserved;
    int64_t m_e;
} pf_report_t;
int pf_report(pf_plan_t *plan, const uint64_t *d_idx, uint32_t n, const uint32_t *d_n, pf_report_t *d_out,
              void *stream);

#ifdef __cplusplus
}
#endif
#endif
