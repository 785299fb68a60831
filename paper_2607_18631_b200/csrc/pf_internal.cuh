// pf_internal.cuh -- device-side plan description, handle layout and block top-k utilities shared by the
// translation units of libplanfront.so.  Nothing here is part of the public ABI.
#pragma once

#include <cuda_runtime.h>
#include <utility>
#include <stdint.h>

#include "planfront.h"
#include "planfront_bench.h"   // timing classes of the measurement hooks

namespace pf {

constexpr int kThreads = 256;        // threads per block of the scoring kernel
constexpr int kTopkCap = 2048;       // shared-memory candidate buffer per block (2 * PF_K_MAX)
constexpr uint32_t kSlabMax = 16384; // upper bound on candidates per slab (inner-axis product)
constexpr int kInnerVals = 1024;     // inner-axis values the scoring kernel keeps in shared memory
constexpr int kOrderMaxSlabs = 1 << 20;  // calls with more slabs visit them by a permutation instead of an order table
constexpr int kTailFillsPerBlock = 4;    // constant-fill slabs per block kept, at least, for the end of the visiting order
constexpr int kFillsPerEvaluated = 3;    // fills interleaved per evaluated slab at the start of the visiting order (measured: 1: 0.392 ms, 2: 0.384, 3: 0.380, 4: 0.379, 6: 0.382, 8: 0.385, 12: 0.396)
// Inside a search call a kernel of its own streams the constant slabs on the plan's fill stream, from right behind
// the scoring kernel to the end of the call: ONE launch beside the scoring kernel, the selection, the simulator and
// the re-ranking.  The bytes travel as bulk copies issued by one block of kFillThreads threads per SM.  Measured on
// the benchmark's space (ms per step): plain 16-byte stores instead of bulk copies, in two launches of 160 and 96
// threads per SM (more crowd the simulator's shared-memory polling out of the load/store pipe, fewer cannot keep
// HBM busy): 0.529; bulk copies in two launches (one until the simulator's pre-pass is done, one beside the
// simulator kernel): 0.466; in one launch: 0.437 -- whatever the block size (32 .. 256 threads), the number of
// issuing threads (16 .. 128) or the piece size (2 .. 4 KB), but only with a working block on (nearly) every SM,
// which takes a grid of 256 blocks per SM (32 per SM: 42 - 82 SMs covered, 0.55 - 0.58 ms with two launches; 128:
// ~100 SMs, 0.535; 256: 144 - 148 SMs; 512: 148 SMs, no faster).
// Fills interleaved with the evaluated slabs inside the scoring kernel only move time from one kernel to the other.
constexpr int kFillsPerEvaluatedSplit = 0;
constexpr int kFillBlocksPerSm = 1;
constexpr int kFillThreads = 128;      // block size of the fill kernel; every thread issues copies
constexpr int kFillGridPerSm = 256;    // blocks launched per SM; a block works only if it is among the first on its SM
constexpr int kQueueCap = 4096;   // cost-model queue of the scoring kernel (entries), drained when it may fill up

struct DevSched {
    int kind, overlap, mapped;
    float hide_frac, sched_ovh;
    int n_chunks;      // comm chunking for the simulator's two-stream layer timeline (0: use hide_frac)
    float sm_frac;     // SMs held by communication kernels while overlapping
};

struct DevKern {
    uint32_t needs_caps, avail_mask;
    int is_native, wbytes;
    float dtype_mult, patch_ovh;
    float eff[PF_NBUCKET];
    int dtype;
};

// Everything a kernel needs about the plan space except the axis value lists (global memory).
// Passed by value as a __grid_constant__ kernel parameter, so uniform reads come from the constant bank.
struct DevPlan {
    // --- index space
    int phase, n_axes;
    int n_inner;          // axes [0, n_inner) vary inside a slab, the rest select the slab
    int n_pre_rules;      // leading rules that depend on outer axes only (checked once per slab)
    uint32_t slab;        // candidates per slab = product of inner radices (<= kSlabMax)
    uint32_t radix[PF_MAX_AXES];
    uint32_t magic[PF_MAX_AXES];   // ceil(2^32 / radix) for the inner axes: q = umulhi(n, magic)
    int val_off[PF_MAX_AXES];      // offset of each axis' value list in the packed value array
    int wide;                      // 1: rule arithmetic needs 64-bit integers
    int sim_domain_all;            // 1: every feasible candidate lies inside the simulator's domain
    int tab_n[3];                  // per-slab rule table over the inner ones of (sched, mb, v); 0 = not used
    uint32_t slab_mul;             // slabs are visited in the order (s * slab_mul) mod n_slabs
    // --- model (Sec. 3.1) and host-derived per-layer constants
    int L, H, nh, nkv, hd, attn_kind, kv_latent, rope_dim, E, K, F, S, Fs, seq, vocab;
    int wb, gb, ob, ab, count_embeddings;
    int dk;
    long long P_attn, P_rt, P_e, P_sh, P_dl, P_emb;
    long long a_full, a_sel, a_ckpt;
    int L_dense;                       // leading layers with a plain FFN instead of experts
    long long P_dld, a_full_d, a_sel_d;   // such a layer: parameters that shard by tp, activation bytes per token
    float f_dense_d, f_mlp_d;          // its forward FLOPs per token, and its FFN's share
    float f_dense, f_exp, f_head, f_sh;   // forward FLOPs per token (per layer; head once), rounded to fp32 once
    // --- modeled cluster
    int G;
    uint32_t caps;
    long long budget_bytes, reserved_bytes;
    float peak_flops, hbm_bw, bw_intra, bw_inter, alpha_intra, alpha_inter, bw_host;
    // --- workload
    long long gbs, world;
    int n_scen;
    // --- cost constants, rules, tables
    float eff_dense, bwd_factor, dp_overlap_frac, dualpipe_startup_div, step_overhead, offload_overlap_penalty;
    int ep_scope, layer_mode, tp_max, world_min, world_max, enforce;
    int n_sched, n_kern;
    DevSched sched[PF_MAX_SCHED];
    DevKern kern[PF_MAX_KERN];
    // --- calibration domain of the constants
    int dom_attached, dom_gpu, dom_m_lo, dom_m_hi, gpu_id;
    uint32_t dom_dtypes;
    // --- the checked build's record (PF_BOUNDS_CHECK): word 0 = bits of the sites that saw an index outside its
    // array, word 1 = the last such site, words 2-3 = the offending index, words 4-5 = the array's length
    unsigned int *chk;
};

// Index checks of the checked build (-DPF_BOUNDS_CHECK; the ordinary build compiles them away).  PF_AT(i, n, site)
// is the index to use for an array of n elements: i itself when 0 <= i < n; otherwise the violation is recorded in
// the plan's check record and 0 is used instead, so the access stays inside the array and nothing traps.
enum {
    PF_SITE_ORDER = 0, PF_SITE_IMAGE = 1, PF_SITE_QUEUE = 2, PF_SITE_TABLE = 3, PF_SITE_PASS = 4, PF_SITE_INFO = 5,
    PF_SITE_DENSE = 6, PF_SITE_KEYS = 7, PF_SITE_DIGEST = 8, PF_SITE_VALS = 9, PF_SITE_TIMELINE = 10,
    PF_SITE_DURATION = 11, PF_SITE_RECORD = 12, PF_SITE_SIM_OUT = 13, PF_SITE_DUAL_OPS = 14, PF_SITE_CHUNK = 15,
    PF_SITE_SURVIVOR = 16, PF_SITE_TOPK_BUF = 17, PF_SITE_SCEN = 18
};
#ifdef PF_BOUNDS_CHECK
__device__ __forceinline__ long long check_at(unsigned int *chk, long long i, long long n, int site)
{
    if (i >= 0 && i < n) return i;
    if (chk) {
        atomicOr(chk, 1u << site);
        chk[1] = (unsigned int)site;
        chk[2] = (unsigned int)i;
        chk[3] = (unsigned int)((unsigned long long)i >> 32);
        chk[4] = (unsigned int)n;
        chk[5] = (unsigned int)((unsigned long long)n >> 32);
    }
    return 0;
}
#define PF_AT(chk, i, n, site) pf::check_at((chk), (long long)(i), (long long)(n), (site))
#else
#define PF_AT(chk, i, n, site) (i)
#endif

}  // namespace pf

// The opaque handle of the C ABI.
struct pf_plan {
    pf::DevPlan dev;
    uint64_t size;                 // N
    int device;
    int sm_count;
    // host copies
    int32_t *h_vals;               // packed axis value lists
    int32_t axis_len[PF_MAX_AXES];
    // device buffers owned by the handle: all inside one block (arena) from a per-device cache
    void *arena;
    size_t arena_cap;
    int32_t *d_vals;               // packed axis value lists
    int32_t *d_scen;               // serve: P[n_scen] then O[n_scen]
    // Slab visiting order of the most recent pf_score range (device: 64 header words, order_cap order words,
    // order_cap class bytes); NULL when the space has too many slabs.  The host key below says which range
    // the table was last built for; the device header says which range it actually holds.
    uint32_t *d_order;
    uint32_t order_cap;
    uint64_t order_slab_lo;
    uint32_t order_n_slabs, order_tail, order_fpe;
    // pf_search overlaps three things once the evaluated part of the space has been scored: the reduction of the
    // analytic top-k (side_stream), the streaming of the constant slabs (fill_stream) and, on the caller's stream,
    // the survivor selection and the simulator.  Streams and fork / join events belong to the plan (training
    // plans; created with the plan).
    cudaStream_t side_stream, fill_stream;
    cudaEvent_t ev_fork, ev_join, ev_fork3, ev_fill, ev_count, ev_compact;
    // simulator order tables (built at create for training plans)
    void *sim_tables;
    unsigned int *d_fill_ctl;      // queue head and per-SM block counts of the fill kernels (2 KB)
    unsigned int *d_check;         // the checked build's record (dev.chk); 64 bytes, zero unless a check fired
    // optional per-kernel-class event timing (pf_timing_enable)
    void *timing;
};

namespace pf {

// ------------------------------------------------------------------ error plumbing (host)
void set_cuda_error(cudaError_t e, const char *where);
// PF_OK when the plan's device is the calling thread's current device, PF_EINVAL otherwise (a launch on another
// device would hand its kernels pointers of the plan's device: a fault on the GPU instead of an error code)
int check_device(const pf_plan_t *p);
void count_launch();
// Make sure `kernel` may be launched with `bytes` of dynamic shared memory on the plan's device.  That limit is state
// of the (kernel, device) pair, shared by every thread of the process: it is only ever RAISED, under a lock, so a
// launch that needs less than another plan's call just asked for stays valid (two threads setting it back and
// forth made the smaller setting win now and then: "invalid argument" at the other thread's launch).
cudaError_t ensure_dynamic_smem(const void *kernel, int device, size_t bytes);
// event pair around the launches of one kernel class; no-ops unless pf_timing_enable(plan, 1)
void timing_begin(pf_plan_t *p, int cls, cudaStream_t st);
void timing_end(pf_plan_t *p, int cls, int n_kernels, cudaStream_t st);
#define PF_CUDA_TRY(expr, where)                        \
    do {                                                \
        cudaError_t e__ = (expr);                       \
        if (e__ != cudaSuccess) {                       \
            pf::set_cuda_error(e__, where);             \
            return PF_ECUDA;                            \
        }                                               \
    } while (0)

// ------------------------------------------------------------------ chained launches
// The small kernels of a call form a chain on one stream, each reading what the one before wrote.  A plain launch
// starts only after the kernel before it has completed and its launch has then been processed: a few microseconds
// per link.  A chained launch (programmatic stream serialization) lets the GPU schedule the grid as soon as every
// block of the kernel before it has passed chain_enter() or left, so that the launch itself overlaps that kernel;
// the new grid's blocks then wait in chain_enter() until that kernel has completed and its writes are visible.
// Rule for a kernel launched this way, and for the kernel in front of it: chain_enter() is its first statement
// (nothing before it touches global memory).  In a kernel launched the plain way chain_enter() does nothing.
__device__ __forceinline__ void chain_enter()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

// ------------------------------------------------------------------ keys
// A ranked candidate is one 64-bit key: (fp32 score bits << 32) | (0xFFFFFFFF - rel), rel = position in
// the call's range (< 2^32 - 1).  Scores are positive floats, so unsigned key order = (score descending,
// index ascending) when sorted descending.  Key 0 = empty slot.
__device__ __forceinline__ unsigned long long make_key(float score, uint32_t rel)
{
    return ((unsigned long long)__float_as_uint(score) << 32) | (unsigned long long)(0xFFFFFFFFu - rel);
}
__device__ __forceinline__ float key_score(unsigned long long key) { return __uint_as_float((uint32_t)(key >> 32)); }
__device__ __forceinline__ uint32_t key_rel(unsigned long long key) { return 0xFFFFFFFFu - (uint32_t)key; }

// ------------------------------------------------------------------ block top-k in shared memory
// buf[kTopkCap] holds candidate keys, *count the number of valid ones, *thr the current admission
// threshold (the k-th best key once k are held, else 0).  All functions are block-collective unless
// noted; the block may have any multiple of 32 threads.

// Descending bitonic sort of buf[0, n_sort); n_sort a power of two <= kTopkCap; buf has room for 64 keys at
// least.  PAIRS = kTopkCap / 2 / blockDim.x.  Each thread owns adjacent elements (2p, 2p+1) for its pair
// numbers p = tid, tid + blockDim, ...; a warp therefore owns a 64-element window.  All compare-exchanges
// with stride <= 32 stay inside that window: they run on registers with warp shuffles.  Only the wider
// strides (>= 64) go through shared memory with block barriers.
template <int PAIRS>
__device__ inline void tk_sort_desc(unsigned long long *buf, int n_sort)
{
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    const int n_eff = n_sort < 64 ? 64 : n_sort;   // whole warps take part; missing elements are zeros
    unsigned long long r0[PAIRS], r1[PAIRS];
    __syncthreads();
#pragma unroll
    for (int t = 0; t < PAIRS; t++) {
        const int i0 = 2 * (tid + t * nt);
        r0[t] = i0 < n_sort ? buf[i0] : 0ull;
        r1[t] = i0 + 1 < n_sort ? buf[i0 + 1] : 0ull;
    }
    for (int size = 2; size <= n_eff; size <<= 1) {
        int stride = size >> 1;
        if (stride >= 64) {
#pragma unroll
            for (int t = 0; t < PAIRS; t++) {
                const int i0 = 2 * (tid + t * nt);
                if (i0 < n_eff) {
                    buf[i0] = r0[t];
                    buf[i0 + 1] = r1[t];
                }
            }
            for (; stride >= 64; stride >>= 1) {
                __syncthreads();
                for (int i = tid; i < n_eff / 2; i += nt) {
                    const int lo = 2 * i - (i & (stride - 1)), hi = lo + stride;
                    const bool desc = (lo & size) == 0;
                    const unsigned long long a = buf[lo], b = buf[hi];
                    if (desc ? (a < b) : (a > b)) {
                        buf[lo] = b;
                        buf[hi] = a;
                    }
                }
            }
            __syncthreads();
#pragma unroll
            for (int t = 0; t < PAIRS; t++) {
                const int i0 = 2 * (tid + t * nt);
                if (i0 < n_eff) {
                    r0[t] = buf[i0];
                    r1[t] = buf[i0 + 1];
                }
            }
        }
        for (; stride >= 1; stride >>= 1) {
#pragma unroll
            for (int t = 0; t < PAIRS; t++) {
                const int i0 = 2 * (tid + t * nt);
                if (i0 >= n_eff) continue;   // whole warps only: n_eff / 2 is a multiple of 32
                const bool desc = (i0 & size) == 0;
                if (stride == 1) {
                    const unsigned long long a = r0[t], b = r1[t];
                    if (desc ? (a < b) : (a > b)) {
                        r0[t] = b;
                        r1[t] = a;
                    }
                } else {
                    const int lm = stride >> 1;
                    const unsigned long long o0 = __shfl_xor_sync(0xFFFFFFFFu, r0[t], lm);
                    const unsigned long long o1 = __shfl_xor_sync(0xFFFFFFFFu, r1[t], lm);
                    const bool keep_max = ((lane & lm) == 0) == desc;
                    r0[t] = keep_max ? (r0[t] > o0 ? r0[t] : o0) : (r0[t] < o0 ? r0[t] : o0);
                    r1[t] = keep_max ? (r1[t] > o1 ? r1[t] : o1) : (r1[t] < o1 ? r1[t] : o1);
                }
            }
        }
    }
#pragma unroll
    for (int t = 0; t < PAIRS; t++) {
        const int i0 = 2 * (tid + t * nt);
        if (i0 < n_eff) {
            buf[i0] = r0[t];
            buf[i0 + 1] = r1[t];
        }
    }
    __syncthreads();
}

// Keep the best k: sort what is held (padded to a power of two), clamp the count, refresh the threshold.
template <int PAIRS>
__device__ inline void tk_prune(unsigned long long *buf, int *count, unsigned long long *thr, int k)
{
    __syncthreads();
    int c = *count;
    if (c > kTopkCap) c = kTopkCap;
    int n_sort = 32;
    while (n_sort < c) n_sort <<= 1;
    for (int i = c + threadIdx.x; i < n_sort; i += blockDim.x) buf[i] = 0ull;
    tk_sort_desc<PAIRS>(buf, n_sort);
    if (threadIdx.x == 0) {
        int n = c < k ? c : k;
        *count = n;
        *thr = (n == k) ? buf[k - 1] : 0ull;
    }
    __syncthreads();
}

// Append the block's held keys that are >= min_key (after tk_prune: sorted, c of them) to a compact global
// key list.  s_base: two shared ints of scratch.  Block-collective.
__device__ inline void tk_flush(const unsigned long long *buf, int c, unsigned long long min_key, int *s_base,
                                unsigned long long *out_keys, unsigned int *out_count)
{
    if (threadIdx.x == 0) s_base[1] = 0;
    __syncthreads();
    // the buffer is sorted descending: the cut is the last position whose key is still >= min_key
    for (int i = threadIdx.x; i < c; i += blockDim.x)
        if (buf[i] >= min_key && (i + 1 == c || buf[i + 1] < min_key)) s_base[1] = i + 1;
    __syncthreads();
    const int keep = s_base[1];
    if (threadIdx.x == 0) s_base[0] = keep > 0 ? (int)atomicAdd(out_count, (unsigned int)keep) : 0;
    __syncthreads();
    unsigned long long *out = out_keys + s_base[0];
    for (int i = threadIdx.x; i < keep; i += blockDim.x) out[i] = buf[i];
}

// Append this thread's key if it beats the threshold.  Warp-collective (all 32 lanes must call); the
// caller guarantees room for one key per thread of the block.
__device__ __forceinline__ void tk_push(unsigned long long *buf, int *count, unsigned long long thr, bool has,
                                        unsigned long long key)
{
    bool take = has && key > thr;
    unsigned mask = __ballot_sync(0xFFFFFFFFu, take);
    if (mask == 0) return;
    int lane = threadIdx.x & 31;
    int leader = __ffs(mask) - 1;
    int base = 0;
    if (lane == leader) base = atomicAdd(count, __popc(mask));
    base = __shfl_sync(0xFFFFFFFFu, base, leader);
    if (take) {
        int pos = base + __popc(mask & ((1u << lane) - 1u));
        if (pos < kTopkCap) buf[pos] = key;
    }
}

// What the first pass of the survivor selection would collect, gathered by the scoring kernel instead when the
// two run inside one search call: the coarse / fine histograms of the eligible candidates' score bits, the
// eligible count of every selection chunk, the list of chunks with any, and its length.  All zeroed by the caller.
struct ScoreDigest {
    unsigned int *hist1, *coarse1, *elig, *list, *n_list;
    uint32_t chunk;   // candidates per selection chunk
};

// does the plan's order table hold this range and shape?  (hdr: slab_lo (2 words), n_slabs, tail, head length,
// fills per evaluated slab)
__device__ __forceinline__ bool order_table_valid(const uint32_t *hdr, uint64_t slab_lo, uint32_t n_slabs, uint32_t tail,
                                                  uint32_t fpe)
{
    return hdr[0] == (uint32_t)slab_lo && hdr[1] == (uint32_t)(slab_lo >> 32) && hdr[2] == n_slabs && hdr[3] == tail &&
           hdr[5] == fpe;
}

// While the constant slabs of a scoring call are still being streamed out, a reader of the dense outputs may
// only trust the slabs the scoring kernel itself has written: the evaluated ones (class byte 0).  cls == NULL: no
// fill is in flight, everything may be read.  The class bytes count only while the order table they were made
// with is the one the scoring call used (otherwise that call's scoring kernel wrote every slab itself).
struct FillGuard {
    const uint8_t *cls = nullptr;
    const uint32_t *hdr = nullptr;
    uint64_t slab_lo = 0;
    uint32_t n_slabs = 0, slab = 1, tail = 0, fpe = 0;
};

// What the kernel that streams the constant slabs behind the head of the visiting order needs (pf_score.cu).
struct FillArgs {
    uint64_t first, count, slab_lo;
    uint32_t n_slabs, slab, order_tail, order_fpe;
    uint8_t *reason;
    float *tput;
    long long *mem;
    const uint32_t *order, *order_hdr;
    // the queue of constant slabs and the per-SM registration of the kernel's blocks (plan-owned, zeroed per call)
    unsigned int *ticket, *sm_slots;
    unsigned int *done;            // counts the slabs the launch has filled
    uint32_t per_sm;               // working blocks per SM
    uint32_t piece, issuers;       // zeros travel as bulk copies of `piece` bytes, issued by the first `issuers` threads
    unsigned int *chk;             // the checked build's record (unused otherwise)
};

// How a scoring call may spread over the plan's streams (all off: one stream, one scoring kernel).
//   topk_aside: the key-list reduction runs on side_stream; ev_join is recorded when it is done.
//   fill_aside: the scoring kernel visits the evaluated slabs only (plus `fills_per_evaluated` constant ones each);
//               the remaining constant slabs are left to a second, lean kernel that is started on fill_stream
//               right behind the scoring kernel; ev_fill is recorded when that is done.
// The caller makes its stream wait for the events it was told were recorded (*joined bits) before it touches
// the workspace (ev_join) or lets the call's results count as complete (ev_fill).
struct ScoreSpread {
    bool topk_aside = false, fill_aside = false;
    int fills_per_evaluated = kFillsPerEvaluated;
    bool join_pending = false, fill_pending = false;   // out: events the caller still has to wait for
    FillGuard guard;                                   // out: set when fill_pending
};
// pf_compact's launches on `st`; guard: class bytes to trust instead of constant blocks still in flight (or NULL)
int compact_run(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
                const int64_t *d_mem, uint64_t *d_hist, uint8_t *d_mask, pf_record_t *d_records, uint64_t record_cap,
                uint64_t *d_n_feasible, void *d_workspace, cudaStream_t st, const FillGuard *guard);
// after compact_run on the same stream and workspace: the feasibility bits of the chunks that hold a feasible plan
// only, to a device-visible address (mapped host memory included); the rest of the mask is zero and not written
int compact_mask_run(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason, uint8_t *mask,
                     void *d_workspace, cudaStream_t st, const FillGuard *guard);
int simulate_run(pf_plan_t *p, const uint64_t *d_surv_idx, uint64_t n, const uint64_t *d_n, uint32_t jitter_seed,
                 float *d_tput_sim, uint8_t *d_sim_status, uint32_t k, uint64_t *d_topk_idx, float *d_topk_score,
                 uint32_t *d_topk_count, void *d_workspace, size_t workspace_bytes, cudaStream_t st);

// internal entry points behind pf_score / pf_select_survivors (dg / have_digest: the fused search call)
int score_run(pf_plan_t *p, uint64_t first, uint64_t count, uint8_t *d_reason, float *d_tput, int64_t *d_mem,
              uint32_t k, uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count, void *d_workspace,
              size_t workspace_bytes, cudaStream_t st, const ScoreDigest *dg, ScoreSpread *spread);
int select_clear(pf_plan_t *p, uint64_t count, void *d_workspace, size_t workspace_bytes, cudaStream_t st,
                 ScoreDigest *dg_out);
int select_run(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
               uint64_t s_max, uint64_t *d_surv_idx, uint64_t *d_surv_count, void *d_workspace,
               size_t workspace_bytes, cudaStream_t st, bool have_digest, const FillGuard *guard);

// host: workspace layout of one top-k reduction whose producers append at most n_keys_max keys in total.
// ctrl is 256 bytes: uint32 [0] producer work counter, [1] keys in list A, [2] keys in list B, [3] spare;
// uint64 at byte 16: the producers' shared admission threshold (largest k-th key any block has reached).
constexpr int kReduceSeg = 2048;     // keys one block of the reduce kernel walks through
constexpr int kReduceThreads = 1024;
constexpr int kFastKeys = 16384;     // a key list up to this long is sorted whole by the final reduce block
struct TopkLayout {
    size_t off_ctrl, off_keys_a, off_keys_b, total;
};
inline TopkLayout topk_layout(uint64_t n_keys_max, uint32_t k)
{
    TopkLayout l;
    size_t kk = k ? k : 1;
    if (n_keys_max < kk) n_keys_max = kk;
    l.off_ctrl = 0;
    l.off_keys_a = 256;
    size_t a = ((size_t)n_keys_max * 8 + 255) & ~(size_t)255;
    // the second list: what pass 1 of the reduction leaves -- at most k keys from each of at most kFastKeys / k
    // blocks, and never more keys than went in (the older, larger bound is kept so that workspace sizes stay put)
    size_t blocks = (n_keys_max + kReduceSeg - 1) / kReduceSeg;
    size_t keys_b = blocks * kk;
    const size_t short_list = n_keys_max < (size_t)kFastKeys ? (size_t)n_keys_max : (size_t)kFastKeys;
    if (keys_b < short_list) keys_b = short_list;
    size_t b = (keys_b * 8 + 255) & ~(size_t)255;
    l.off_keys_b = l.off_keys_a + a;
    l.total = l.off_keys_b + b;
    return l;
}

// host: reduce a compact key list (device count in ctrl[1], at most n_keys_max keys) to the final outputs.
// idx_map (device, may be NULL): final index = idx_map[rel] instead of first + rel.
// Returns the number of kernels launched through *n_kernels.  chained: the kernel that wrote the list is the operation
// right before this call on the same stream (the first launch here is then a chained one).
int launch_topk_reduce(void *d_workspace, const TopkLayout &lay, uint64_t n_keys_max, uint32_t k, uint64_t first,
                       const uint64_t *d_idx_map, uint64_t *d_topk_idx, float *d_topk_score, uint32_t *d_topk_count,
                       cudaStream_t st, int *n_kernels, bool chained = false);

// host: top-k of a dense score array (entries with score <= 0 are skipped; ties go to the lower position).
// The workspace is laid out by dense_topk_layout; idx_map as in launch_topk_reduce.
struct DenseTopkLayout {
    int blocks;
    uint64_t keys_max;
    TopkLayout tk;
};
DenseTopkLayout dense_topk_layout(int sm_count, uint64_t n, uint32_t k);
int launch_dense_topk(const float *d_score, uint64_t n, const uint64_t *d_n, uint32_t k, const uint64_t *d_idx_map,
                      void *d_workspace, const DenseTopkLayout &lay, uint64_t *d_topk_idx, float *d_topk_score,
                      uint32_t *d_topk_count, cudaStream_t st, int *n_kernels, bool ctrl_cleared = false);
// (ctrl_cleared: the caller has zeroed the first 256 bytes of the layout's control block earlier on the stream, so
// that no memset stands between the kernel that wrote the scores and this one's first, chained, launch)

}  // namespace pf
