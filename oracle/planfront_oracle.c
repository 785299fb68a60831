/*
 * planfront_oracle.c -- see planfront_oracle.h.  TEST INFRASTRUCTURE ONLY.
 *
 * One candidate at a time, in the order the paper gives for its predicate (Sec. 3.3, Fig. 2):
 * decode -> structural divisibility checks -> emit dry-run rules -> memory gate -> analytic
 * step time (Sec. 3.2) -> realization tax (Sec. 3.2) -> score.  No blocking, no fusion, no
 * reordering.  Integers are int64, floating quantities are double.
 */
#include "planfront_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ op tally (-DORACLE_COUNT_OPS)
 *
 * The counting build charges, block by block, the arithmetic, comparison and logic operators that
 * the definition writes out (loads, stores and assignments are free; a ceil-division is 3 integer
 * ops, a highest-set-bit search 4).  A block's operators are charged when control reaches it, so a
 * candidate rejected by rule r pays for decode and rules 1..r only.  The totals give the
 * algorithmic operation count per candidate for an ALU roofline; they change no result. */
#ifdef ORACLE_COUNT_OPS
static _Thread_local int64_t tl_ops_i, tl_ops_f, tl_ops_n;
static int64_t g_ops_i, g_ops_f, g_ops_n;
#define OPS(i, f) (tl_ops_i += (i), tl_ops_f += (f))
#else
#define OPS(i, f) ((void)0)
#endif

int orc_ops_enabled(void)
{
#ifdef ORACLE_COUNT_OPS
    return 1;
#else
    return 0;
#endif
}

void orc_ops_reset(void)
{
#ifdef ORACLE_COUNT_OPS
    g_ops_i = g_ops_f = g_ops_n = 0;
#endif
}

/* out[0] integer ops, out[1] floating ops, out[2] candidates evaluated since the last reset */
void orc_ops_read(int64_t out[3])
{
#ifdef ORACLE_COUNT_OPS
    out[0] = g_ops_i; out[1] = g_ops_f; out[2] = g_ops_n;
#else
    out[0] = out[1] = out[2] = 0;
#endif
}

/* ------------------------------------------------------------------ helpers */

static int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
static int64_t imin(int64_t a, int64_t b) { return a < b ? a : b; }
static int64_t imax(int64_t a, int64_t b) { return a > b ? a : b; }

/* position of the highest set bit, x >= 1 */
static int flog2(int64_t x)
{
    int r = 0;
    while (x > 1) {
        x >>= 1;
        r++;
    }
    return r;
}

/* smallest c with 2^c >= n, n >= 1 */
static int clog2(int64_t n)
{
    int c = 0;
    while (((int64_t)1 << c) < n) c++;
    return c;
}

/* tokens-per-expert bucket: 8 power-of-two buckets over the calibration domain [64, 8192]
 * (Appendix, "Testbeds and calibration domains"): <128, 128.., 256.., ..., 4096.., >=8192 */
static int me_bucket(int64_t m_e)
{
    int b = flog2(imax(m_e, 1)) - 6;
    if (b < 0) b = 0;
    if (b > 7) b = 7;
    return b;
}

int64_t orc_budget_bytes(int64_t hbm_bytes)
{
    /* Sec. 2.1: 72 GB budget = 80 GB HBM at a 0.9 usable fraction */
    return hbm_bytes * 9 / 10;
}

/* ------------------------------------------------------------------ model constants */

void orc_derive(const orc_model_t *m, orc_derived_t *d)
{
    const int64_t H = m->H, nh = m->nh, nkv = m->nkv, hd = m->hd, ab = m->ab;
    const int64_t hq = m->hd_q > 0 ? m->hd_q : hd;
    memset(d, 0, sizeof(*d));
    d->dk = m->attn_kind ? m->kv_latent + m->rope_dim : hd;
    if (m->attn_kind == 0) {
        /* q, k, v, o projections */
        d->P_attn = H * nh * hq + 2 * H * nkv * hd + nh * hd * H;
    } else {
        /* q proj, compressed kv (+ rope) down-proj, kv up-proj, o proj */
        d->P_attn = H * nh * hq + H * (m->kv_latent + m->rope_dim) + m->kv_latent * nh * 2 * hd + nh * hd * H;
    }
    d->P_rt = H * m->E;                      /* router */
    d->P_e = m->n_mats * H * m->F;           /* one routed expert */
    d->P_sh = m->S * m->n_mats * H * m->Fs;  /* shared experts */
    d->P_dl = d->P_attn + d->P_sh;           /* dense params per layer that shard by tp */
    d->P_emb = m->count_embeddings ? m->vocab * H : 0;

    int64_t qkv_act = m->attn_kind == 0 ? (nh + 2 * nkv) * hd
                                        : nh * hd + m->kv_latent + m->rope_dim + 2 * nh * hd;
    /* activation bytes per token per layer: ln1 input, qkv-proj input, q/k/v, o-proj input */
    d->a_attn = ab * (2 * H + qkv_act + nh * hd);
    /* ln2 input, router input, fp32 router logits, K dispatched copies, combine output */
    d->a_fix = ab * (2 * H) + 4 * m->E + ab * m->K * H + ab * H;
    /* gate, up, act*up for routed copies and shared experts */
    d->a_ffn = ab * 3 * (m->K * m->F + m->S * m->Fs);
    d->a_full = d->a_attn + d->a_fix + d->a_ffn;
    d->a_sel = d->a_attn + d->a_fix;
    d->a_ckpt = ab * H;

    /* forward FLOPs per token per layer; causal attention core = 4*seq*nh*dk / 2 */
    d->f_attn = 2 * d->P_attn + 2 * m->seq * nh * d->dk;
    d->f_rt = 2 * H * m->E;
    d->f_sh = 2 * d->P_sh;
    d->f_dense = d->f_attn + d->f_rt + d->f_sh;
    d->f_exp = 2 * m->K * d->P_e;
    d->f_head = 2 * m->vocab * H;

    /* a leading dense layer: attention + a plain FFN (gate, up, down of width F_dense), no router, no experts */
    d->P_dld = d->P_attn + m->n_mats * H * m->F_dense;
    d->a_sel_d = d->a_attn + ab * (2 * H);              /* ln2 input, FFN input */
    d->a_full_d = d->a_sel_d + ab * 3 * m->F_dense;     /* gate, up, act*up */
    d->f_mlp_d = 2 * m->n_mats * H * m->F_dense;
    d->f_dense_d = d->f_attn + d->f_mlp_d;
}

uint64_t orc_space_size(const orc_problem_t *pb)
{
    uint64_t n = 1;
    for (int a = 0; a < pb->axes.n_axes; a++) n *= (uint64_t)pb->axes.len[a];
    return n;
}

/* mixed-radix decode, least-significant axis first (Sec. 3.1: one tuple carries every knob) */
static void decode(const orc_axes_t *ax, uint64_t idx, int64_t *value)
{
    uint64_t rem = idx;
    OPS(2 * ax->n_axes, 0); /* one mod and one div per axis */
    for (int a = 0; a < ax->n_axes; a++) {
        uint64_t n = (uint64_t)ax->len[a];
        uint64_t digit = rem % n;
        rem = rem / n;
        value[a] = ax->val[a][digit];
    }
}

/* Which parts of the calibration domain a query falls outside of (principle P4): 0 = inside, or no domain */
static int64_t domain_why(const orc_problem_t *pb, const orc_kern_t *kn, int64_t m_e)
{
    const orc_domain_t *dm = &pb->domain;
    int64_t why = 0;
    if (!dm->attached) return 0;
    if (dm->gpu_id >= 0 && dm->gpu_id != pb->cluster.gpu_id) why |= ORC_WHY_GPU;
    if (((dm->dtype_mask >> kn->dtype) & 1) == 0) why |= ORC_WHY_DTYPE;
    if (m_e < dm->m_lo) why |= ORC_WHY_M_LOW;
    if (m_e > dm->m_hi) why |= ORC_WHY_M_HIGH;
    return why;
}

/* ------------------------------------------------------------------ alpha-beta collectives */

typedef struct {
    double bw, alpha;
} link_t;

static link_t link_of(const orc_cluster_t *c, int64_t span)
{
    link_t l;
    if (span <= c->G) {
        l.bw = c->bw_intra;
        l.alpha = c->alpha_intra;
    } else {
        l.bw = c->bw_inter;
        l.alpha = c->alpha_inter;
    }
    return l;
}

/* all-reduce; reduce-scatter + all-gather has the same alpha-beta form */
static double t_allreduce(int64_t n, double bytes, link_t lk)
{
    if (n <= 1) return 0.0;
    return 2.0 * (double)(n - 1) / (double)n * bytes / lk.bw + 2.0 * (double)clog2(n) * lk.alpha;
}
/* all-gather of `bytes` (the gathered size); a reduce-scatter has the same alpha-beta form */
static double t_allgather(int64_t n, double bytes, link_t lk)
{
    if (n <= 1) return 0.0;
    return (double)(n - 1) / (double)n * bytes / lk.bw + (double)clog2(n) * lk.alpha;
}
static double t_alltoall(int64_t n, double bytes, link_t lk)
{
    if (n <= 1) return 0.0;
    return (double)(n - 1) / (double)n * bytes / lk.bw + lk.alpha;
}

/* ------------------------------------------------------------------ training candidate */

static int eval_train(const orc_problem_t *pb, const orc_derived_t *dv, uint64_t idx, orc_detail_t *o)
{
    const orc_model_t *M = &pb->model;
    const orc_cluster_t *C = &pb->cluster;
    const orc_rules_t *R = &pb->rules;
    const orc_consts_t *K0 = &pb->consts;
    int64_t val[ORC_MAX_AXES] = {0};
    decode(&pb->axes, idx, val);
    int64_t kv = val[0], rec = val[1], s = val[2], mb = val[3], v = val[4];
    int64_t ep = val[5], pp = val[6], tp = val[7], dp = val[8], world = val[9];
    /* the sharding dimension is orthogonal to the layout and defaults to zero1 (Sec. 3.1) */
    int64_t shard = pb->axes.n_axes > 10 ? val[10] : ORC_SHARD_ZERO1;
    o->kv = kv; o->rec = rec; o->sched = s; o->mb = mb; o->v = v;
    o->ep = ep; o->pp = pp; o->tp = tp; o->shard = shard;

    /* rule 1 WORLD: data parallelism is derived from the world size (Sec. 3.1) unless both are
     * enumerated, in which case the product must match; whole nodes beyond one node */
    OPS(dp == 0 ? 15 : 10, 0);
    if (dp == 0) {
        if (world % (tp * pp) != 0) return o->reason = ORC_R_WORLD;
        dp = world / (tp * pp);
    }
    if (world == 0) world = tp * pp * dp;
    o->dp = dp; o->world = world;
    if (tp * pp * dp != world) return o->reason = ORC_R_WORLD;
    if (world < R->world_min || world > R->world_max) return o->reason = ORC_R_WORLD;
    if (world > C->G && world % C->G != 0) return o->reason = ORC_R_WORLD;

    /* rule 2 TP: tensor degrees over the head-divisible subset (Sec. 3.3) */
    OPS(10, 0);
    if (tp > R->tp_max || tp > C->G || M->nh % tp != 0) return o->reason = ORC_R_TP;
    if (M->S > 0 && M->Fs % tp != 0) return o->reason = ORC_R_TP;
    if (R->ep_scope == 0 && M->F % tp != 0) return o->reason = ORC_R_TP;

    /* rule 3 EP: expert degrees over the admissible divisors; EP inside DP (Sec. 4) or inside DP*TP */
    OPS(R->ep_scope ? 6 : 5, 0);
    if (M->E % ep != 0) return o->reason = ORC_R_EP;
    if (R->ep_scope == 0) {
        if (dp % ep != 0) return o->reason = ORC_R_EP;
    } else {
        if ((dp * tp) % ep != 0) return o->reason = ORC_R_EP;
    }

    /* rule 4 BATCH */
    OPS(3, 0);
    if (pb->workload.gbs % (dp * mb) != 0) return o->reason = ORC_R_BATCH;

    OPS(6 + 3, 0); /* derived integers, then rule 5 */
    int64_t kind = pb->sched[s].kind, ov = pb->sched[s].overlap;
    int64_t v_eff = (v == 0) ? (kind == ORC_KIND_INTERLEAVED ? 2 : 1) : v;
    int64_t m = pb->workload.gbs / (dp * mb);
    int64_t t = mb * M->seq;
    int64_t Q = pp * v_eff;
    o->kind = kind; o->ov = ov; o->v_eff = v_eff; o->m = m; o->t = t; o->Q = Q;

    /* rule 5 VSTAGE */
    if (kind == ORC_KIND_INTERLEAVED) {
        if (v_eff < 2 || pp < 2) return o->reason = ORC_R_VSTAGE;
    } else {
        if (v_eff != 1) return o->reason = ORC_R_VSTAGE;
    }

    /* rule 6 LAYERS: layer count vs pipeline depth (Fig. 2: 27 mod pp*v != 0) */
    OPS(3 + 4, 0); /* the rule, then Lc and Ls */
    if (R->layer_mode == 0) {
        if (M->L % Q != 0) return o->reason = ORC_R_LAYERS;
    } else {
        if (Q > M->L) return o->reason = ORC_R_LAYERS;
    }
    int64_t Lc = cdiv(M->L, Q);
    int64_t Ls = v_eff * Lc; /* layers on the bottleneck rank */
    o->Lc = Lc; o->Ls = Ls;
    /* leading dense layers on the first rank (it holds virtual stages 0, pp, 2pp, ...) and on the last one:
     * stage q covers layers [q*Lc, (q+1)*Lc) */
    int64_t nd0 = 0, nd_last = 0;
    for (int64_t c = 0; c < v_eff; c++) {
        nd0 += imax(0, imin(Lc, M->L_dense - c * pp * Lc));
        nd_last += imax(0, imin(Lc, M->L_dense - (c * pp + pp - 1) * Lc));
    }
    o->nd0 = nd0; o->nd_last = nd_last;

    /* rule 7 MICROBATCH: what each static schedule order needs to be well formed */
    OPS(kind == ORC_KIND_1F1B ? 2 : kind == ORC_KIND_INTERLEAVED ? 3 : 8, 0);
    if (kind == ORC_KIND_INTERLEAVED) {
        if (m % pp != 0) return o->reason = ORC_R_MICROBATCH;
    } else if (kind == ORC_KIND_DUALPIPE) {
        if (m % 2 != 0) return o->reason = ORC_R_MICROBATCH;
        if (pp > 1 && pp % 2 != 0) return o->reason = ORC_R_MICROBATCH;
    }

    /* rule 8 KERNEL_MISSING: variant needs a capability the cluster lacks, or the autotune
     * report has no entry at this expert shape (Sec. 3.3 kernel tier) */
    OPS(5 + 4 + 4 + 6, 0); /* group sizes, m_e, its bucket, the two table tests */
    int64_t tps = R->ep_scope ? tp : 1;
    int64_t etp = R->ep_scope ? 1 : tp;
    int64_t edp = R->ep_scope ? dp * tp / ep : dp / ep;
    int64_t m_e = (t * M->K * ep) / (M->E * tps);
    int b = me_bucket(m_e);
    o->edp = edp; o->m_e = m_e; o->bucket = b;
    const orc_kern_t *kn = &pb->kern[kv];
    if ((kn->needs_caps & ~C->caps) != 0) return o->reason = ORC_R_KERNEL_MISSING;
    if (((kn->avail_mask >> b) & 1) == 0) return o->reason = ORC_R_KERNEL_MISSING;

    /* rules 9, 10: the emit dry-run (Sec. 4 "Emitters"); skipped in unconstrained mode (Sec. 3.3) */
    OPS(R->enforce_realizability ? 8 : 1, 0);
    if (R->enforce_realizability) {
        if (!pb->sched[s].mapped) return o->reason = ORC_R_UNMAPPED_SCHEDULE;
        if (ov && (rec == ORC_REC_FULL || (kind == ORC_KIND_1F1B && pp > 1)))
            return o->reason = ORC_R_OVERLAP_PRECOND;
    }

    /* ---- memory (bytes on rank 0, which holds the most in-flight activations) ---- */
    OPS(3 + 6 + 7 + 7 + 4 + 9 + 2 + 4 + 6 + 1 + 5, 0); /* pm, emb, N_dense, N_exp, w+g, o, A_tok, A_layer, units,
                                                          bytes_a, sum and gate */
    if (rec == ORC_REC_FULL) OPS(6, 0);
    if (pb->axes.n_axes > 10) OPS(val[10] == ORC_SHARD_FSDP ? 16 : 4, val[10] == ORC_SHARD_FSDP ? 22 : val[10] ? 4 : 0);
    if ((pp == 1 || kind == ORC_KIND_DUALPIPE) && M->count_embeddings) OPS(9, 0);
    int64_t pm = (kind == ORC_KIND_DUALPIPE && pp > 1) ? 2 : 1; /* two stage copies per rank */
    int64_t emb = cdiv(dv->P_emb, tp) * ((pp == 1 || kind == ORC_KIND_DUALPIPE) ? 2 : 1);
    /* the rank's MoE layers (both stage copies of a DualPipe-style rank; its second copy sits at the far end of
     * the pipeline and has no leading dense layer) and its leading dense layers */
    int64_t n_moe = pm * Ls - nd0;
    int64_t N_dense = n_moe * (cdiv(dv->P_dl, tp) + dv->P_rt) + nd0 * cdiv(dv->P_dld, tp) + emb;
    int64_t N_exp = n_moe * (M->E / ep) * cdiv(dv->P_e, etp);
    int64_t bytes_w = M->wb * (N_dense + N_exp);
    int64_t bytes_g = M->gb * (N_dense + N_exp);
    /* distributed optimizer: dense shard over dp, expert shard over the expert-DP group
     * (Sec. 5 RQ1: the expert optimizer state is ep-invariant) */
    int64_t n_shard = cdiv(N_dense, dp) + cdiv(N_exp, edp); /* parameters whose state this rank owns */
    int64_t bytes_o_dense = M->ob * cdiv(N_dense, dp);
    int64_t bytes_o_expert = M->ob * cdiv(N_exp, edp);
    int64_t bytes_o = bytes_o_dense + bytes_o_expert;
    int64_t bytes_buf = 0;
    if (shard == ORC_SHARD_ZERO1_OFFLOAD) {
        /* the optimizer state lives in host memory */
        bytes_o_dense = bytes_o_expert = bytes_o = 0;
    } else if (shard == ORC_SHARD_FSDP) {
        /* parameters and gradients are sharded like the optimizer state; the all-gather working buffer
         * (boundary B7 of the paper's catalogue) holds the unsharded parameters of the layer in use and of
         * the one being prefetched */
        bytes_w = M->wb * n_shard;
        bytes_g = M->gb * n_shard;
        int64_t P_layer = cdiv(dv->P_dl, tp) + dv->P_rt + (M->E / ep) * cdiv(dv->P_e, etp);
        bytes_buf = imin(2, pm * Ls) * M->wb * P_layer;
    }
    int64_t A_tok = rec == ORC_REC_NONE ? dv->a_full : rec == ORC_REC_SELECTIVE ? dv->a_sel : dv->a_ckpt;
    int64_t A_tok_d = rec == ORC_REC_NONE ? dv->a_full_d : rec == ORC_REC_SELECTIVE ? dv->a_sel_d : dv->a_ckpt;
    int64_t A_layer = cdiv(t * A_tok, tp);
    int64_t A_layer_d = cdiv(t * A_tok_d, tp);
    /* activation bytes of one microbatch across the rank's Ls layers */
    int64_t A_rank = (Ls - nd0) * A_layer + nd0 * A_layer_d;
    int64_t bytes_a;
    if (kind == ORC_KIND_1F1B)
        bytes_a = imin(pp, m) * A_rank;
    else if (kind == ORC_KIND_INTERLEAVED) /* chunks in flight, each a v-th of the rank's layers */
        bytes_a = imin(pp * v_eff + pp - 1, m * v_eff) * A_rank / v_eff;
    else
        bytes_a = imin(pp + 1, m) * A_rank;
    if (rec == ORC_REC_FULL) bytes_a += cdiv(t * dv->a_full, tp); /* the layer being recomputed */
    if ((pp == 1 || kind == ORC_KIND_DUALPIPE) && M->count_embeddings)
        bytes_a += 4 * cdiv(t * M->vocab, tp); /* fp32 logits where the head lives */
    int64_t mem = bytes_w + bytes_g + bytes_o + bytes_buf + bytes_a + C->reserved_bytes;
    o->N_dense = N_dense; o->N_exp = N_exp; o->bytes_w = bytes_w; o->bytes_g = bytes_g;
    o->bytes_o_dense = bytes_o_dense; o->bytes_o_expert = bytes_o_expert; o->bytes_o = bytes_o;
    o->bytes_a = bytes_a; o->bytes_buf = bytes_buf; o->mem = mem;

    /* rule 11 MEMORY: the gate rejects when the peak exceeds the budget (Sec. 5 RQ1: 79.39 > 72) */
    if (mem > C->budget_bytes) return o->reason = ORC_R_MEMORY;

    /* ---- analytic step time ---- */
    /* compute 4+5+1+1, recompute <= 7, TP all-reduce 10 (+6 int), all-to-all 8 (+4 int), exposure 7,
     * per-layer sums 8, head 4, stage sums 7, p2p <= 4 (+2 int), closed form <= 10 (+4 int),
     * gradient all-reduces 20 (+12 int), optimizer 2, step 5, throughput and prices 7 (+3 int), flag 2 int */
    OPS(6 + 4 + 2 + 4 + 12 + 3 + 2, 4 + 5 + 1 + 1 + 7 + 10 + 8 + 7 + 8 + 4 + 7 + 4 + 10 + 20 + 2 + 5 + 7);
    double td = (double)t, tpd = (double)tp;
    double peak = C->peak_flops;
    double cD = td * (double)dv->f_dense / (tpd * peak * K0->eff_dense);
    double cE = td * (double)dv->f_exp / (tpd * peak * kn->dtype_mult * kn->eff[b]);
    double cF = cD + cE;
    double cB = K0->bwd_factor * cF;
    double rc;
    if (rec == ORC_REC_NONE)
        rc = 0.0;
    else if (rec == ORC_REC_SELECTIVE)
        rc = (2.0 / 3.0) * (cE + td * (double)dv->f_sh / (tpd * peak * K0->eff_dense));
    else
        rc = cF;
    double tpc = 2.0 * t_allreduce(tp, (double)(M->ab * t * M->H), link_of(C, tp));
    double a2a = 2.0 * t_alltoall(ep, (double)(M->ab * t * M->K * M->H) / tpd, link_of(C, tp * ep));
    /* the hiding benefit is conditioned out in the offload domain (Sec. 5 RQ2) */
    double h = (ov && shard != ORC_SHARD_ZERO1_OFFLOAD) ? pb->sched[s].hide_frac : 0.0;
    double xF = a2a - fmin(h * a2a, cF);
    double xB = a2a - fmin(h * a2a, cB + rc);
    double F_l = cF + tpc + xF;
    double B_l = cB + rc + tpc + xB + (rec == ORC_REC_FULL ? tpc + xF : 0.0);
    double headF = td * (double)dv->f_head / (tpd * peak * K0->eff_dense);
    /* a leading dense layer: no experts, no all-to-all */
    double cDd = td * (double)dv->f_dense_d / (tpd * peak * K0->eff_dense);
    double rcd = rec == ORC_REC_NONE ? 0.0
                 : rec == ORC_REC_SELECTIVE ? (2.0 / 3.0) * td * (double)dv->f_mlp_d / (tpd * peak * K0->eff_dense)
                                            : cDd;
    double F_ld = cDd + tpc;
    double B_ld = K0->bwd_factor * cDd + rcd + tpc + (rec == ORC_REC_FULL ? tpc : 0.0);
    /* the closed forms take the slower of the two extreme ranks: the first (most leading dense layers) and the
     * last (fewest) */
    double F0 = (double)(Ls - nd0) * F_l + (double)nd0 * F_ld, B0 = (double)(Ls - nd0) * B_l + (double)nd0 * B_ld;
    double F1 = (double)(Ls - nd_last) * F_l + (double)nd_last * F_ld;
    double B1 = (double)(Ls - nd_last) * B_l + (double)nd_last * B_ld;
    int first_slower = F0 + B0 > F1 + B1;
    double F = (first_slower ? F0 : F1) + headF / (double)pp;
    double B = (first_slower ? B0 : B1) + K0->bwd_factor * headF / (double)pp;
    double p = 0.0;
    if (pp > 1) {
        link_t lw = link_of(C, world);
        p = (double)(M->ab * t * M->H) / tpd / lw.bw + lw.alpha;
    }
    double T_pipe;
    if (kind == ORC_KIND_1F1B)
        T_pipe = (double)(m + pp - 1) * (F + B) + 2.0 * (double)(pp - 1) * p;
    else if (kind == ORC_KIND_INTERLEAVED)
        T_pipe = ((double)m + (double)(pp - 1) / (double)v_eff) * (F + B) + 2.0 * (double)(Q - 1) * p;
    else
        T_pipe = (double)m * (F + B) + (double)imax(pp - 2, 0) * B + (F + B) / K0->dualpipe_startup_div +
                 2.0 * (double)(pp - 1) * p;
    link_t ldp = link_of(C, tp * dp);
    double T_dp = t_allreduce(dp, (double)((M->gb + M->wb) * N_dense), ldp) +
                  t_allreduce(edp, (double)((M->gb + M->wb) * N_exp), ldp);
    double T_opt = 2.0 * (double)bytes_o / C->hbm_bw;
    if (shard == ORC_SHARD_ZERO1_OFFLOAD) {
        /* the step runs on the host: the shard's gradients go down and its updated weights come back */
        T_opt = (double)((M->gb + M->wb) * n_shard) / C->bw_host;
    } else if (shard == ORC_SHARD_FSDP) {
        /* per microbatch the parameters are gathered for the forward and again for the backward pass and the
         * gradients are reduce-scattered; this replaces the gradient all-reduce of the replicated regimes */
        double ag = t_allgather(dp, (double)(M->wb * N_dense), ldp) + t_allgather(edp, (double)(M->wb * N_exp), ldp);
        double rs = t_allgather(dp, (double)(M->gb * N_dense), ldp) + t_allgather(edp, (double)(M->gb * N_exp), ldp);
        T_dp = (double)m * (2.0 * ag + rs);
    }
    double T_step = T_pipe + (1.0 - K0->dp_overlap_frac) * T_dp + T_opt + K0->step_overhead;

    /* ---- pricing: throughput / (1 + frac) on the plans that take the taxed path ---- */
    double tput = (double)(pb->workload.gbs * M->seq) / (T_step * (double)world);
    o->tput_unpriced = tput;
    if (!kn->is_native) tput = tput / (1.0 + kn->patch_ovh);
    if (ov) tput = tput / (1.0 + pb->sched[s].sched_ovh);
    /* the contention penalty prices exactly the offloaded-and-overlapped plans (Sec. 3.2) */
    if (ov && shard == ORC_SHARD_ZERO1_OFFLOAD) tput = tput / (1.0 + K0->offload_overlap_penalty);

    o->cF = cF; o->cB = cB; o->rc = rc; o->tpc = tpc; o->a2a = a2a; o->xF = xF; o->xB = xB;
    o->F_l = F_l; o->B_l = B_l; o->headF = headF; o->F = F; o->B = B; o->p = p;
    o->F_ld = F_ld; o->B_ld = B_ld; o->cD = cD; o->cE = cE;
    o->T_pipe = T_pipe; o->T_dp = T_dp; o->T_opt = T_opt; o->T_step = T_step; o->tput = tput;

    int reason = ORC_FEASIBLE;
    o->why = domain_why(pb, kn, m_e);
    if (o->why) reason |= ORC_FLAG_EXTRAPOLATED;
    return o->reason = reason;
}

/* ------------------------------------------------------------------ serving candidate */

static int eval_serve(const orc_problem_t *pb, const orc_derived_t *dv, uint64_t idx, orc_detail_t *o)
{
    const orc_model_t *M = &pb->model;
    const orc_cluster_t *C = &pb->cluster;
    const orc_consts_t *K0 = &pb->consts;
    int64_t val[ORC_MAX_AXES] = {0};
    decode(&pb->axes, idx, val);
    int64_t kv = val[0], Cc = val[1], Bd = val[2], dpa = val[3], ep = val[4], tp = val[5], sc = val[6];
    int64_t world = pb->workload.world;
    int64_t P = pb->workload.scen_P[sc], O = pb->workload.scen_O[sc];
    o->kv = kv; o->chunk = Cc; o->batch = Bd; o->dpa = dpa; o->ep = ep; o->tp = tp; o->scen = sc;
    o->world = world;

    /* rule 1 WORLD: dp-attention needs dp == ep with the real world size (Sec. 2.1, boundary B5);
     * without it experts shard inside the tensor-parallel world, ep*moe_dp == tp (Sec. 4) */
    OPS(2 + 4, 0);
    if (world % tp != 0) return o->reason = ORC_R_WORLD;
    if (dpa) {
        if (world / tp != ep || ep < 2) return o->reason = ORC_R_WORLD;
    } else {
        if (tp % ep != 0) return o->reason = ORC_R_WORLD;
    }
    /* rule 2 TP */
    OPS(4 + 3, 0); /* the rule, then engine sizes */
    if (tp > C->G || M->nh % tp != 0) return o->reason = ORC_R_TP;
    int64_t n_eng = dpa ? tp * ep : tp;
    int64_t moe_tp = n_eng / ep;
    /* rule 3 EP */
    OPS(5, 0);
    if (M->E % ep != 0 || M->F % moe_tp != 0) return o->reason = ORC_R_EP;
    /* rule 4 BATCH */
    OPS(3 + 1, 0);
    if (dpa && Bd % ep != 0) return o->reason = ORC_R_BATCH;
    int64_t b_loc = dpa ? Bd / ep : Bd;

    /* rule 8 KERNEL_MISSING: decode and prefill expert shapes both need an entry */
    OPS(4 + 8 + 3 + 7, 0); /* two shapes, two buckets, capability test, two table tests */
    int64_t m_e = (Bd * M->K) / M->E;
    int64_t m_ep = (Cc * M->K) / M->E;
    int b = me_bucket(m_e), b_pre = me_bucket(m_ep);
    o->m_e = m_e; o->bucket = b; o->bucket_pre = b_pre;
    const orc_kern_t *kn = &pb->kern[kv];
    if ((kn->needs_caps & ~C->caps) != 0) return o->reason = ORC_R_KERNEL_MISSING;
    if (((kn->avail_mask >> b) & 1) == 0 || ((kn->avail_mask >> b_pre) & 1) == 0)
        return o->reason = ORC_R_KERNEL_MISSING;

    /* ---- memory: weights + KV cache + prefill activation workspace ---- */
    OPS(19 + 6 + 5 + 3 + 3 + 1, 0); /* weights, KV bytes per token, cache, workspace, sum, gate */
    /* leading dense layers (DeepSeek-style stacks): attention + a plain FFN sharded by tp, no router, no experts */
    int64_t Ld = M->L_dense, Lm = M->L - M->L_dense;
    if (Ld > 0) OPS(6, 30);
    int64_t w = Lm * (cdiv(dv->P_dl, tp) * M->wb + dv->P_rt * M->wb +
                      (M->E / ep) * cdiv(dv->P_e, moe_tp) * kn->wbytes) +
                Ld * cdiv(dv->P_dld, tp) * M->wb + 2 * cdiv(M->vocab * M->H, tp) * M->wb;
    /* the MLA latent is replicated across tensor-parallel ranks */
    int64_t kv_tok = M->attn_kind ? (M->kv_latent + M->rope_dim) * M->ab : cdiv(2 * M->nkv * M->hd, tp) * M->ab;
    int64_t kvc = b_loc * (P + O) * M->L * kv_tok;
    int64_t act = 8 * M->ab * Cc * M->H;
    int64_t mem = w + kvc + act + C->reserved_bytes;
    o->bytes_w = w; o->bytes_a = act; o->mem = mem;
    if (mem > C->budget_bytes) return o->reason = ORC_R_MEMORY;

    /* ---- time: per-layer max(compute, HBM) + collectives; decode at mean context ---- */
    /* decode step: context and weight terms 9, experts touched 5, attention 14, experts 8, collective <= 11,
     * layer sum 4; prefill: chunking 2 (+3 int), experts touched 6, attention 13, experts 8, collective <= 11,
     * sum 5; throughput and price 8, flag 2 int; plus ~10 int in operand products and collective shapes */
    OPS(1 + 3 + 2 + 10, 9 + 5 + 14 + 8 + 11 + 4 + 2 + 6 + 13 + 8 + 11 + 5 + 8);
    link_t lk = link_of(C, n_eng);
    double peak = C->peak_flops, hbm = C->hbm_bw, effd = K0->eff_dense;
    double tpd = (double)tp, nen = (double)n_eng, bl = (double)b_loc, dk = (double)dv->dk;
    double nh = (double)M->nh;
    double ctx = (double)P + (double)O / 2.0;
    double attn_w = (double)(dv->P_dl * M->wb) / tpd;
    double e_per = (double)(M->E / ep);
    double exp_unit = (double)(dv->P_e * kn->wbytes) / (double)moe_tp;
    /* experts touched: between one and all local experts, growing with routed copies */
    double xd = (double)(Bd * M->K) / (double)ep;
    double exp_w_d = fmin(e_per, fmax(1.0, xd)) * exp_unit;
    double t_attn_d = fmax(bl * (2.0 * (double)dv->P_dl + 4.0 * ctx * nh * dk) / (tpd * peak * effd),
                           (attn_w + bl * ctx * (double)kv_tok) / hbm);
    double t_moe_d = fmax((double)Bd * (double)dv->f_exp / (nen * peak * kn->dtype_mult * kn->eff[b]),
                          exp_w_d / hbm);
    double t_com_d = dpa ? 2.0 * t_alltoall(n_eng, (double)M->ab * bl * (double)(M->K * M->H), lk)
                         : 2.0 * t_allreduce(tp, (double)(M->ab * Bd * M->H), lk);
    /* a leading dense layer: its weights (attention + FFN) stream once per step, its FLOPs are 2 per parameter and
     * token plus the attention core, and its two tensor-parallel all-reduces carry the tokens of this attention
     * group; no all-to-all */
    double t_dl_d = 0.0, t_dl_p = 0.0;
    double w_dl = (double)(dv->P_dld * M->wb) / tpd;
    link_t ltp = link_of(C, tp);
    if (Ld > 0)
        t_dl_d = fmax(bl * (2.0 * (double)dv->P_dld + 4.0 * ctx * nh * dk) / (tpd * peak * effd),
                      (w_dl + bl * ctx * (double)kv_tok) / hbm) +
                 2.0 * t_allreduce(tp, (double)M->ab * bl * (double)M->H, ltp);
    double T_dec = (double)Lm * (t_attn_d + t_moe_d + t_com_d) + (double)Ld * t_dl_d + K0->step_overhead;
    int64_t nc = cdiv(P, Cc);
    double c = (double)P / (double)nc;
    double xp = c * (double)M->K / (double)ep;
    double exp_w_p = fmin(e_per, fmax(1.0, xp)) * exp_unit;
    double t_attn_p = fmax(c * (2.0 * (double)dv->P_dl + 4.0 * ((double)P / 2.0) * nh * dk) / (tpd * peak * effd),
                           attn_w / hbm);
    double t_moe_p = fmax(c * (double)dv->f_exp / (nen * peak * kn->dtype_mult * kn->eff[b_pre]),
                          exp_w_p / hbm);
    double t_com_p = dpa ? 2.0 * t_alltoall(n_eng, (double)M->ab * c * (double)(M->K * M->H), lk)
                         : 2.0 * t_allreduce(tp, (double)M->ab * c * (double)M->H, lk);
    if (Ld > 0)
        t_dl_p = fmax(c * (2.0 * (double)dv->P_dld + 4.0 * ((double)P / 2.0) * nh * dk) / (tpd * peak * effd), w_dl / hbm) +
                 2.0 * t_allreduce(tp, (double)M->ab * c * (double)M->H, ltp);
    double T_pre = (double)nc * ((double)Lm * (t_attn_p + t_moe_p + t_com_p) + (double)Ld * t_dl_p);
    double tput = (double)(Bd * O) / (bl * T_pre + (double)O * T_dec) / nen;
    o->tput_unpriced = tput;
    if (!kn->is_native) tput = tput / (1.0 + kn->patch_ovh);
    o->T_dec = T_dec; o->T_pre = T_pre; o->tput = tput;

    int reason = ORC_FEASIBLE;
    o->why = domain_why(pb, kn, m_e);
    if (o->why) reason |= ORC_FLAG_EXTRAPOLATED;
    return o->reason = reason;
}

static int eval_one(const orc_problem_t *pb, uint64_t idx, orc_detail_t *detail)
{
    orc_detail_t local;
    orc_derived_t dv;
    if (!detail) detail = &local;
    memset(detail, 0, sizeof(*detail));
    orc_derive(&pb->model, &dv);
    int r = pb->workload.phase == 0 ? eval_train(pb, &dv, idx, detail) : eval_serve(pb, &dv, idx, detail);
    if ((r & 0x7f) != 0) detail->tput = 0.0;
#ifdef ORACLE_COUNT_OPS
    tl_ops_n++;
#endif
    return r;
}

/* add the calling thread's tally to the totals */
static void ops_fold(void)
{
#ifdef ORACLE_COUNT_OPS
    __atomic_fetch_add(&g_ops_i, tl_ops_i, __ATOMIC_RELAXED);
    __atomic_fetch_add(&g_ops_f, tl_ops_f, __ATOMIC_RELAXED);
    __atomic_fetch_add(&g_ops_n, tl_ops_n, __ATOMIC_RELAXED);
    tl_ops_i = tl_ops_f = tl_ops_n = 0;
#endif
}

int orc_eval(const orc_problem_t *pb, uint64_t idx, orc_detail_t *detail)
{
    int r = eval_one(pb, idx, detail);
    ops_fold();
    return r;
}

int orc_score_range(const orc_problem_t *pb, uint64_t first, uint64_t count, uint8_t *reason,
                    double *tput, int64_t *mem, int n_threads)
{
    int used = 1;
    if (n_threads < 1) n_threads = 1;
#ifdef _OPENMP
#pragma omp parallel num_threads(n_threads)
    {
#pragma omp single
        used = omp_get_num_threads();
#pragma omp for schedule(static)
        for (int64_t i = 0; i < (int64_t)count; i++) {
            orc_detail_t d;
            int r = eval_one(pb, first + (uint64_t)i, &d);
            if (reason) reason[i] = (uint8_t)r;
            if (tput) tput[i] = d.tput;
            if (mem) mem[i] = d.mem;
        }
        ops_fold();
    }
#else
    for (uint64_t i = 0; i < count; i++) {
        orc_detail_t d;
        int r = eval_one(pb, first + i, &d);
        if (reason) reason[i] = (uint8_t)r;
        if (tput) tput[i] = d.tput;
        if (mem) mem[i] = d.mem;
    }
    ops_fold();
#endif
    return used;
}

/* ------------------------------------------------------------------ top-k by full sort */

typedef struct {
    double score;
    uint64_t idx;
} ranked_t;

static int cmp_ranked(const void *a, const void *b)
{
    const ranked_t *x = (const ranked_t *)a, *y = (const ranked_t *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    if (x->idx < y->idx) return -1;
    if (x->idx > y->idx) return 1;
    return 0;
}
static int cmp_u64(const void *a, const void *b)
{
    uint64_t x = *(const uint64_t *)a, y = *(const uint64_t *)b;
    return x < y ? -1 : x > y ? 1 : 0;
}

uint64_t orc_topk(const uint8_t *reason, const double *tput, uint64_t first, uint64_t count,
                  uint64_t k, uint64_t *out_idx, double *out_score)
{
    uint64_t nf = 0;
    for (uint64_t i = 0; i < count; i++)
        if ((reason[i] & 0x7f) == 0) nf++;
    ranked_t *r = (ranked_t *)malloc((nf ? nf : 1) * sizeof(ranked_t));
    uint64_t j = 0;
    for (uint64_t i = 0; i < count; i++)
        if ((reason[i] & 0x7f) == 0) {
            r[j].score = tput[i];
            r[j].idx = first + i;
            j++;
        }
    qsort(r, nf, sizeof(ranked_t), cmp_ranked);
    uint64_t n = nf < k ? nf : k;
    for (uint64_t i = 0; i < n; i++) {
        out_idx[i] = r[i].idx;
        out_score[i] = r[i].score;
    }
    free(r);
    return n;
}

uint64_t orc_topk_list(const uint64_t *idx, const double *score, uint64_t n, uint64_t k,
                       uint64_t *out_idx, double *out_score)
{
    ranked_t *r = (ranked_t *)malloc((n ? n : 1) * sizeof(ranked_t));
    for (uint64_t i = 0; i < n; i++) {
        r[i].score = score[i];
        r[i].idx = idx[i];
    }
    qsort(r, n, sizeof(ranked_t), cmp_ranked);
    uint64_t w = n < k ? n : k;
    for (uint64_t i = 0; i < w; i++) {
        out_idx[i] = r[i].idx;
        out_score[i] = r[i].score;
    }
    free(r);
    return w;
}

/* simulator domain: training plans with pp <= 32 ranks and at most 8 virtual stages per rank */
static int in_sim_domain(const orc_problem_t *pb, uint64_t idx)
{
    if (pb->workload.phase != 0) return 0;
    int64_t val[ORC_MAX_AXES] = {0};
    decode(&pb->axes, idx, val);
    int64_t s = val[2], v = val[4], pp = val[6];
    int64_t kind = pb->sched[s].kind;
    int64_t v_eff = (v == 0) ? (kind == ORC_KIND_INTERLEAVED ? 2 : 1) : v;
    return pp <= ORC_MAX_RANKS && v_eff <= ORC_MAX_V;
}

uint64_t orc_select_survivors(const orc_problem_t *pb, const uint8_t *reason, const double *tput,
                              uint64_t first, uint64_t count, uint64_t s_max, uint64_t *out_idx)
{
    uint64_t nf = 0;
    for (uint64_t i = 0; i < count; i++)
        if ((reason[i] & 0x7f) == 0 && in_sim_domain(pb, first + i)) nf++;
    ranked_t *r = (ranked_t *)malloc((nf ? nf : 1) * sizeof(ranked_t));
    uint64_t j = 0;
    for (uint64_t i = 0; i < count; i++)
        if ((reason[i] & 0x7f) == 0 && in_sim_domain(pb, first + i)) {
            r[j].score = tput[i];
            r[j].idx = first + i;
            j++;
        }
    qsort(r, nf, sizeof(ranked_t), cmp_ranked);
    uint64_t n = nf < s_max ? nf : s_max;
    for (uint64_t i = 0; i < n; i++) out_idx[i] = r[i].idx;
    qsort(out_idx, n, sizeof(uint64_t), cmp_u64);
    free(r);
    return n;
}

/* ------------------------------------------------------------------ serving: per-plan aggregate */

uint64_t orc_serve_plan_count(const orc_problem_t *pb)
{
    const orc_axes_t *ax = &pb->axes;
    return orc_space_size(pb) / (uint64_t)ax->len[ax->n_axes - 1];
}

void orc_aggregate_serving(const orc_problem_t *pb, const uint8_t *reason, const double *tput,
                           uint8_t *plan_reason, double *plan_tput)
{
    const orc_axes_t *ax = &pb->axes;
    const int64_t n_scen = ax->len[ax->n_axes - 1];
    const uint64_t n_plans = orc_serve_plan_count(pb);
    for (uint64_t p = 0; p < n_plans; p++) {
        int first_fail = 0, flags = 0;
        double tokens = 0.0, time = 0.0;
        for (int64_t i = 0; i < n_scen; i++) {
            uint64_t idx = p + n_plans * (uint64_t)i;
            int r = reason[idx];
            if ((r & 0x7f) != 0) {
                if (!first_fail) first_fail = r & 0x7f;
                continue;
            }
            flags |= r & ORC_FLAG_EXTRAPOLATED;
            double O = (double)pb->workload.scen_O[ax->val[ax->n_axes - 1][i]];
            tokens += O;          /* output tokens of one request of this scenario */
            time += O / tput[idx]; /* and the GPU-seconds they take at this scenario's rate */
        }
        if (first_fail) {
            plan_reason[p] = (uint8_t)first_fail;
            plan_tput[p] = 0.0;
        } else {
            plan_reason[p] = (uint8_t)flags;
            plan_tput[p] = tokens / time;
        }
    }
}

/* ------------------------------------------------------------------ schedule orders */

static int order_1f1b(int pp, int m, int32_t *out, int stride)
{
    for (int s = 0; s < pp; s++) {
        int32_t *o = out + (size_t)s * stride;
        int n = 0;
        int w = pp - s - 1 < m ? pp - s - 1 : m; /* warm-up forwards */
        for (int j = 0; j < w; j++) o[n++] = ORC_OP(s, j, 0, 0);
        for (int i = 0; i < m - w; i++) { /* steady state: one forward, one backward */
            o[n++] = ORC_OP(s, w + i, 0, 0);
            o[n++] = ORC_OP(s, i, 0, 1);
        }
        for (int i = m - w; i < m; i++) o[n++] = ORC_OP(s, i, 0, 1); /* cool-down */
    }
    return 2 * m;
}

/* unit k of rank s -> (virtual stage, microbatch); forward units walk chunks upward,
 * backward units walk them downward; microbatches advance in groups of pp */
static int32_t interleaved_unit(int pp, int v, int s, int k, int isb)
{
    int g = k / (pp * v), r = k % (pp * v);
    int j = g * pp + r % pp;
    int c = isb ? v - 1 - r / pp : r / pp;
    return ORC_OP(c * pp + s, j, 0, isb);
}

static int order_interleaved(int pp, int v, int m, int32_t *out, int stride)
{
    if (m % pp != 0) return -1;
    int U = m * v;
    for (int s = 0; s < pp; s++) {
        int32_t *o = out + (size_t)s * stride;
        int n = 0;
        int w = 2 * (pp - s - 1) + (v - 1) * pp;
        if (w > U) w = U;
        for (int k = 0; k < w; k++) o[n++] = interleaved_unit(pp, v, s, k, 0);
        for (int i = 0; i < U - w; i++) {
            o[n++] = interleaved_unit(pp, v, s, w + i, 0);
            o[n++] = interleaved_unit(pp, v, s, i, 1);
        }
        for (int i = U - w; i < U; i++) o[n++] = interleaved_unit(pp, v, s, i, 1);
    }
    return 2 * U;
}

/*
 * DualPipe-style bidirectional order.  Two directions, each carrying m/2 microbatches through
 * positions 0..pp-1; direction 0 position q lives on rank q, direction 1 on rank pp-1-q.  The
 * per-rank order is DEFINED as what this integer list scheduling produces with nominal durations
 * F = 1, B = 2 ticks and zero latency: at each event time every idle rank starts, among its
 * unstarted ops whose dependencies have finished (and, for a forward at position q, while fewer
 * than pp - q microbatches of that direction are in flight on the rank), the one with the
 * smallest (ready time, backward first, microbatch, direction).
 */
static int order_dualpipe(int pp, int m, int32_t *out, int stride)
{
    if (m % 2 != 0 || (pp > 1 && pp % 2 != 0)) return -1;
    int n = m / 2;
    int total = 4 * n * pp; /* (2 directions) x pp x n x (F, B) */
    /* nominal end times, -1 = not started; index [isb][dir][q][j] */
    int *nend = (int *)malloc(sizeof(int) * (size_t)total);
    for (int i = 0; i < total; i++) nend[i] = -1;
#define NE(isb, d, q, j) nend[((((isb) * 2 + (d)) * pp + (q)) * n) + (j)]
    int busy[ORC_MAX_RANKS], cnt[ORC_MAX_RANKS], inflight[ORC_MAX_RANKS][2];
    if (pp > ORC_MAX_RANKS) {
        free(nend);
        return -1;
    }
    for (int r = 0; r < pp; r++) busy[r] = 0, cnt[r] = 0, inflight[r][0] = inflight[r][1] = 0;
    int started = 0, now = 0;
    while (started < total) {
        for (int r = 0; r < pp; r++) {
            if (busy[r] > now) continue;
            int have = 0, b_ready = 0, b_isb = 0, b_j = 0, b_d = 0, b_q = 0;
            for (int d = 0; d < 2; d++) {
                int q = d == 0 ? r : pp - 1 - r;
                for (int isb = 0; isb < 2; isb++)
                    for (int j = 0; j < n; j++) {
                        if (NE(isb, d, q, j) >= 0) continue;
                        int ready = 0, ok = 1;
                        if (!isb) {
                            if (q > 0) {
                                int e = NE(0, d, q - 1, j);
                                if (e < 0 || e > now) ok = 0;
                                ready = e;
                            }
                            if (inflight[r][d] >= pp - q) ok = 0;
                        } else {
                            int e = NE(0, d, q, j);
                            if (e < 0 || e > now) ok = 0;
                            ready = e;
                            if (q < pp - 1) {
                                int e2 = NE(1, d, q + 1, j);
                                if (e2 < 0 || e2 > now) ok = 0;
                                if (e2 > ready) ready = e2;
                            }
                        }
                        if (!ok) continue;
                        /* key (ready, B before F, j, d) */
                        int better = 0;
                        if (!have) better = 1;
                        else if (ready != b_ready) better = ready < b_ready;
                        else if (isb != b_isb) better = isb > b_isb;
                        else if (j != b_j) better = j < b_j;
                        else better = d < b_d;
                        if (better) have = 1, b_ready = ready, b_isb = isb, b_j = j, b_d = d, b_q = q;
                    }
            }
            if (!have) continue;
            int dur = b_isb ? 2 : 1;
            NE(b_isb, b_d, b_q, b_j) = now + dur;
            busy[r] = now + dur;
            out[(size_t)r * stride + cnt[r]++] = ORC_OP(b_q, b_j, b_d, b_isb);
            if (b_isb) inflight[r][b_d]--; else inflight[r][b_d]++;
            started++;
        }
        /* jump to the next nominal completion */
        int next = -1;
        for (int r = 0; r < pp; r++)
            if (busy[r] > now && (next < 0 || busy[r] < next)) next = busy[r];
        if (next < 0) {
            if (started < total) {
                free(nend);
                return -2; /* no rank busy and nothing ready: the definition deadlocked */
            }
            break;
        }
        now = next;
    }
#undef NE
    free(nend);
    return 2 * m; /* each rank: 2 positions x n microbatches x (F, B) */
}

int orc_schedule_order(int kind, int pp, int v, int m, int32_t *out, int stride)
{
    if (pp < 1 || m < 1) return -1;
    if (kind == ORC_KIND_1F1B) return order_1f1b(pp, m, out, stride);
    if (kind == ORC_KIND_INTERLEAVED) return order_interleaved(pp, v, m, out, stride);
    if (kind == ORC_KIND_DUALPIPE) return order_dualpipe(pp, m, out, stride);
    return -1;
}

/* ------------------------------------------------------------------ evaluating a fixed order */

static int rank_of(int kind, int pp, int q, int dir)
{
    if (kind == ORC_KIND_DUALPIPE) return dir == 0 ? q : pp - 1 - q;
    return q % pp;
}

/*
 * end(op) = max(end of the rank's previous op, max over dependencies (end(dep) + latency)) + duration
 * F(q,j) needs F(q-1,j); B(q,j) needs F(q,j) and B(q+1,j); a dependency on another rank costs p.
 * Also returns, through work_max (may be NULL), max over ranks of the per-microbatch work W_r.
 */
static double eval_order(int kind, int pp, int v, int m, const double *Fq, const double *Bq, double p,
                         double *work_max)
{
    int Q = kind == ORC_KIND_DUALPIPE ? pp : pp * v;
    int nj = kind == ORC_KIND_DUALPIPE ? m / 2 : m;
    int nops_max = 2 * m * (kind == ORC_KIND_INTERLEAVED ? v : 1);
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)pp * nops_max);
    int nops = orc_schedule_order(kind, pp, v, m, order, nops_max);
    if (nops < 0) {
        free(order);
        return -1.0;
    }
    size_t ne = (size_t)2 * 2 * Q * nj;
    double *end = (double *)malloc(sizeof(double) * ne);
    for (size_t i = 0; i < ne; i++) end[i] = -1.0;
#define EN(isb, d, q, j) end[((((size_t)(isb) * 2 + (d)) * Q + (q)) * nj) + (j)]
    int ptr[ORC_MAX_RANKS];
    double last[ORC_MAX_RANKS];
    for (int r = 0; r < pp; r++) ptr[r] = 0, last[r] = 0.0;
    double makespan = 0.0;
    int remaining = pp * nops;
    while (remaining > 0) {
        int progress = 0;
        for (int r = 0; r < pp; r++) {
            while (ptr[r] < nops) {
                int32_t op = order[(size_t)r * nops_max + ptr[r]];
                int isb = ORC_OP_ISB(op), d = ORC_OP_DIR(op), q = ORC_OP_Q(op), j = ORC_OP_J(op);
                double start = last[r];
                if (!isb) {
                    if (q > 0) {
                        double e = EN(0, d, q - 1, j);
                        if (e < 0.0) break;
                        double lat = rank_of(kind, pp, q - 1, d) != r ? p : 0.0;
                        if (e + lat > start) start = e + lat;
                    }
                } else {
                    double e = EN(0, d, q, j);
                    if (e < 0.0) break;
                    if (e > start) start = e;
                    if (q < Q - 1) {
                        double e2 = EN(1, d, q + 1, j);
                        if (e2 < 0.0) break;
                        double lat = rank_of(kind, pp, q + 1, d) != r ? p : 0.0;
                        if (e2 + lat > start) start = e2 + lat;
                    }
                }
                double fin = start + (isb ? Bq[q] : Fq[q]);
                EN(isb, d, q, j) = fin;
                last[r] = fin;
                if (fin > makespan) makespan = fin;
                ptr[r]++;
                remaining--;
                progress = 1;
            }
        }
        if (!progress) {
            makespan = -1.0; /* stalled: the order is not executable */
            break;
        }
    }
#undef EN
    if (work_max) {
        double wm = 0.0;
        for (int r = 0; r < pp; r++) {
            double w = 0.0;
            if (kind == ORC_KIND_DUALPIPE) {
                w = 0.5 * ((Fq[r] + Bq[r]) + (Fq[pp - 1 - r] + Bq[pp - 1 - r]));
            } else {
                int vv = kind == ORC_KIND_INTERLEAVED ? v : 1;
                for (int c = 0; c < vv; c++) w += Fq[c * pp + r] + Bq[c * pp + r];
            }
            if (w > wm) wm = w;
        }
        *work_max = wm;
    }
    free(end);
    free(order);
    return makespan;
}

double orc_makespan(int kind, int pp, int v, int m, const double *Fq, const double *Bq, double p)
{
    if (kind != ORC_KIND_INTERLEAVED) v = 1;
    return eval_order(kind, pp, v, m, Fq, Bq, p, NULL);
}

/* ------------------------------------------------------------------ jitter */

uint32_t orc_mix32(uint32_t x)
{
    x ^= x >> 16;
    x *= 0x7feb352du;
    x ^= x >> 15;
    x *= 0x846ca68bu;
    x ^= x >> 16;
    return x;
}

/* +-10% multiplicative jitter on a stage duration, a pure function of (seed, candidate, stage, F/B) */
double orc_jitter(uint32_t seed, uint64_t idx, int q, int is_backward)
{
    uint32_t h = orc_mix32(seed + 0x9e3779b9u);
    h = orc_mix32(h ^ (uint32_t)(idx & 0xffffffffu));
    h = orc_mix32(h ^ (uint32_t)(idx >> 32));
    h = orc_mix32(h ^ (uint32_t)(2 * q + (is_backward ? 1 : 0)));
    double u = (double)(h >> 8) * (1.0 / 16777216.0);
    return 0.9 + 0.2 * u;
}

/* ------------------------------------------------------------------ two-stream layer timeline */

/* Generic list scheduling over a small op DAG: every op has a stream, a duration and up to two predecessors;
 * a stream that is free starts, among its ops whose predecessors are done, the one that became ready first
 * (ties: lower op number).  Returns the time the last op ends. */
typedef struct {
    int stream, dep0, dep1; /* dep = -1: none */
    double dur;
} ts_op_t;

static double list_schedule(const ts_op_t *op, int n_ops, int n_streams)
{
    double end[64], free_at[4] = {0.0, 0.0, 0.0, 0.0};
    int done[64] = {0};
    int left = n_ops;
    double makespan = 0.0;
    while (left > 0) {
        /* the op that can start earliest over all streams; its start = max(stream free, ready) */
        int best = -1;
        double best_start = 0.0, best_ready = 0.0;
        for (int s = 0; s < n_streams; s++) {
            /* this stream's pick: earliest ready time, then lowest number */
            int pick = -1;
            double pick_ready = 0.0;
            for (int i = 0; i < n_ops; i++) {
                if (done[i] || op[i].stream != s) continue;
                if ((op[i].dep0 >= 0 && !done[op[i].dep0]) || (op[i].dep1 >= 0 && !done[op[i].dep1])) continue;
                double ready = 0.0;
                if (op[i].dep0 >= 0) ready = end[op[i].dep0];
                if (op[i].dep1 >= 0 && end[op[i].dep1] > ready) ready = end[op[i].dep1];
                if (pick < 0 || ready < pick_ready) {
                    pick = i;
                    pick_ready = ready;
                }
            }
            if (pick < 0) continue;
            double start = free_at[s] > pick_ready ? free_at[s] : pick_ready;
            if (best < 0 || start < best_start || (start == best_start && pick < best)) {
                best = pick;
                best_start = start;
                best_ready = pick_ready;
            }
        }
        (void)best_ready;
        if (best < 0) return -1.0; /* cyclic input: cannot happen for the layer DAG */
        end[best] = best_start + op[best].dur;
        free_at[op[best].stream] = end[best];
        done[best] = 1;
        if (end[best] > makespan) makespan = end[best];
        left--;
    }
    return makespan;
}

double orc_two_stream_layer(double A, double e_tot, double d_tot, double c_tot, int n)
{
    ts_op_t op[64];
    if (n < 1) n = 1;
    if (n > 16) n = 16;
    int k = 0;
    op[k++] = (ts_op_t){0, -1, -1, A};                                    /* op 0: the dense part */
    for (int i = 0; i < n; i++) op[k++] = (ts_op_t){1, 0, -1, d_tot / n}; /* ops 1..n: dispatch chunks */
    for (int i = 0; i < n; i++)                                           /* ops n+1..2n: expert chunks, in order */
        op[k++] = (ts_op_t){0, 1 + i, i ? n + i : -1, e_tot / n};
    for (int i = 0; i < n; i++) op[k++] = (ts_op_t){1, n + 1 + i, -1, c_tot / n}; /* combine chunks */
    return list_schedule(op, k, 2);
}

/* ------------------------------------------------------------------ simulator tier */

int orc_simulate(const orc_problem_t *pb, uint64_t idx, uint32_t seed, double *tput_sim, double *T_pipe_sim)
{
    orc_detail_t d;
    int r = orc_eval(pb, idx, &d);
    if (T_pipe_sim) *T_pipe_sim = 0.0;
    if ((r & 0x7f) != 0) {
        *tput_sim = 0.0;
        return ORC_SIM_UNSUPPORTED;
    }
    if (pb->workload.phase != 0 || d.pp > ORC_MAX_RANKS || d.v_eff > ORC_MAX_V) {
        *tput_sim = d.tput; /* outside the simulator's domain: keep the analytic score */
        return ORC_SIM_UNSUPPORTED;
    }
    const orc_model_t *M = &pb->model;
    const orc_consts_t *K0 = &pb->consts;
    int kind = (int)d.kind, pp = (int)d.pp, v = (int)d.v_eff;
    int Q = kind == ORC_KIND_DUALPIPE ? pp : pp * v;
    double Fq[ORC_MAX_RANKS * ORC_MAX_V], Bq[ORC_MAX_RANKS * ORC_MAX_V];
    /* Per-layer times of a MoE layer.  Where the schedule overlaps and says how (comm chunking, SM budget), the
     * exposed communication comes from the two-stream timeline of the layer instead of the alpha-table's hidden
     * fraction: compute is slowed by the SMs the communication kernels hold, the all-to-all halves are the
     * dispatch and the combine, backward splits its compute like forward. */
    const orc_sched_t *sc = &pb->sched[d.sched];
    double F_l = d.F_l, B_l = d.B_l;
    if (d.ov && sc->n_chunks > 0 && d.shard != ORC_SHARD_ZERO1_OFFLOAD) {
        int n = (int)sc->n_chunks;
        double slow = 1.0 / (1.0 - sc->sm_frac);
        double half = 0.5 * d.a2a;
        double fwd = orc_two_stream_layer(d.cD * slow, d.cE * slow, half, half, n);
        double cBt = d.cB + d.rc;                       /* backward compute incl. recompute */
        double share = d.cE / d.cF;                     /* the experts' share of a layer's compute */
        double bwd = orc_two_stream_layer(cBt * (1.0 - share) * slow, cBt * share * slow, half, half, n);
        F_l = d.tpc + fwd;
        B_l = d.tpc + bwd + (d.rec == ORC_REC_FULL ? d.tpc + (fwd - d.cF * slow) : 0.0);
    }
    for (int q = 0; q < Q; q++) {
        /* exact balanced layer split over virtual stages; the head sits on the last one */
        int64_t nq = M->L / Q + (q < M->L % Q ? 1 : 0);
        int64_t start = q * (M->L / Q) + (q < M->L % Q ? q : M->L % Q); /* first layer of the stage */
        int64_t ndq = imax(0, imin(nq, M->L_dense - start));               /* its leading dense layers */
        double f = (double)(nq - ndq) * F_l + (double)ndq * d.F_ld + (q == Q - 1 ? d.headF : 0.0);
        double b = (double)(nq - ndq) * B_l + (double)ndq * d.B_ld + (q == Q - 1 ? K0->bwd_factor * d.headF : 0.0);
        Fq[q] = f * orc_jitter(seed, idx, q, 0);
        Bq[q] = b * orc_jitter(seed, idx, q, 1);
    }
    /* simulated window: at most 64 microbatches (a multiple of pp for the interleaved order) */
    int64_t m = d.m, m_sim = m < ORC_SIM_WINDOW ? m : ORC_SIM_WINDOW;
    if (kind == ORC_KIND_INTERLEAVED) m_sim = (m_sim / pp) * pp;
    double wmax = 0.0;
    double T = eval_order(kind, pp, v, (int)m_sim, Fq, Bq, d.p, &wmax);
    if (T < 0.0) {
        *tput_sim = 0.0;
        return ORC_SIM_STALL;
    }
    /* beyond the window the pipeline is in steady state: the bottleneck rank's work per microbatch */
    if (m > m_sim) T += (double)(m - m_sim) * wmax;
    if (T_pipe_sim) *T_pipe_sim = T;
    double T_step = T + (1.0 - K0->dp_overlap_frac) * d.T_dp + d.T_opt + K0->step_overhead;
    double tput = (double)(pb->workload.gbs * M->seq) / (T_step * (double)d.world);
    if (!pb->kern[d.kv].is_native) tput = tput / (1.0 + pb->kern[d.kv].patch_ovh);
    if (d.ov) tput = tput / (1.0 + pb->sched[d.sched].sched_ovh);
    if (d.ov && d.shard == ORC_SHARD_ZERO1_OFFLOAD) tput = tput / (1.0 + K0->offload_overlap_penalty);
    *tput_sim = tput;
    return ORC_SIM_OK;
}

int orc_simulate_list(const orc_problem_t *pb, const uint64_t *idx, uint64_t n, uint32_t seed,
                      double *tput_sim, uint8_t *status, int n_threads)
{
    int used = 1;
    if (n_threads < 1) n_threads = 1;
#ifdef _OPENMP
#pragma omp parallel num_threads(n_threads)
    {
#pragma omp single
        used = omp_get_num_threads();
#pragma omp for schedule(dynamic, 64)
        for (int64_t i = 0; i < (int64_t)n; i++) {
            double t = 0.0;
            int st = orc_simulate(pb, idx[i], seed, &t, NULL);
            tput_sim[i] = t;
            if (status) status[i] = (uint8_t)st;
        }
    }
#else
    for (uint64_t i = 0; i < n; i++) {
        double t = 0.0;
        int st = orc_simulate(pb, idx[i], seed, &t, NULL);
        tput_sim[i] = t;
        if (status) status[i] = (uint8_t)st;
    }
#endif
    return used;
}
