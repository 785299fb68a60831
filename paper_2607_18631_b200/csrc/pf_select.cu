// pf_select.cu -- survivor selection for the schedule tier (Sec. 3.3: the best analytic candidates are
// refined with the simulator).  Exact top-S by (score descending, index ascending), emitted in ascending
// index order, as a two-level radix select on the fp32 score bits followed by an ordered compaction:
//   hist(hi 16 bits) -> scan -> hist(lo 16 bits inside the threshold bin) -> scan -> per-block counts ->
//   block-offset scan -> ordered write.
// The first pass reads every reason byte with 16-byte loads (a score is touched only where the candidate is
// feasible) and lists the chunks that hold eligible candidates; the later passes visit only those.
#include "pf_internal.cuh"

namespace pf {

constexpr int kSelThreads = 256;
constexpr int kBins = 65536;

// The first eight fields are the public pf_select_cut_t (same order, same widths).
struct SelCtrl {
    unsigned long long total;     // eligible candidates
    unsigned long long above1;    // eligible with hi16 > b1
    unsigned long long n_gt;      // eligible with score bits > threshold
    unsigned long long need_eq;   // how many of the == threshold ones are taken (smallest indices)
    unsigned long long target;    // S
    uint32_t b1, thr_bits;
    int take_all;
    unsigned int n_elig;          // chunks that hold eligible candidates (length of SelArgs::elig_list)
};
static_assert(sizeof(SelCtrl) == sizeof(pf_select_cut_t), "the cut record is the selection's control block");

struct SelArgs {
    uint64_t first, count, s_max;
    const uint8_t *reason;
    const float *tput;
    unsigned int *hist1, *hist2;      // kBins each
    unsigned int *coarse1, *coarse2;  // 256 bins each: sums over groups of 256 fine bins
    unsigned int *blk_elig;           // eligible candidates per chunk, written by the first pass
    unsigned int *elig_list;          // the chunks with blk_elig > 0, in no particular order
    SelCtrl *ctrl;
    unsigned long long *blk_gt, *blk_eq;  // per block counts, then exclusive prefixes
    uint64_t *surv_idx, *surv_count;
    uint64_t chunk;                   // candidates per block (multiple of 16)
    unsigned long long eq_before;     // candidates AT the threshold that lower-ranked shards of the space hold
    FillGuard guard;                  // slabs still being filled by another stream must not be read
};

// class bytes to consult, or NULL when every slab may be read
__device__ __forceinline__ const uint8_t *sel_guard_cls(const SelArgs &A)
{
    const FillGuard &g = A.guard;
    if (!g.cls || !order_table_valid(g.hdr, g.slab_lo, g.n_slabs, g.tail, g.fpe)) return nullptr;
    return g.cls;
}

// eligibility beyond feasibility: the simulator's domain (pp <= 32 ranks, <= 8 virtual stages per rank)
__device__ __forceinline__ bool in_sim_domain(const DevPlan &P, const int32_t *vals, uint64_t idx)
{
    if (P.sim_domain_all) return true;
    int s = 0, v = 0, pp = 0;
    uint64_t rem = idx;
#pragma unroll
    for (int a = 0; a < 7; a++) {
        uint64_t r = P.radix[a];
        uint64_t q = rem / r;
        int d = (int)(rem - q * r);
        rem = q;
        if (a == 2) s = __ldg(vals + P.val_off[2] + d);
        if (a == 4) v = __ldg(vals + P.val_off[4] + d);
        if (a == 6) pp = __ldg(vals + P.val_off[6] + d);
    }
    int v_eff = v == 0 ? (P.sched[s].kind == PF_KIND_INTERLEAVED ? 2 : 1) : v;
    return pp <= PF_SIM_MAX_RANKS && v_eff <= PF_SIM_MAX_V;
}

// 16 reason bytes starting at element e (may run past count: missing ones read as 0xFF = infeasible)
__device__ __forceinline__ uint4 load_reason16(const uint8_t *reason, uint64_t e, uint64_t count)
{
    if (e + 16 <= count && (((uintptr_t)(reason + e)) & 15) == 0) return __ldg(reinterpret_cast<const uint4 *>(reason + e));
    uint32_t w[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
    for (int i = 0; i < 16; i++)
        if (e + i < count) {
            uint32_t b = reason[e + i];
            w[i >> 2] = (w[i >> 2] & ~(0xFFu << (8 * (i & 3)))) | (b << (8 * (i & 3)));
        }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// bit i set: byte i of the 16 has (b & 0x7f) == 0
__device__ __forceinline__ uint32_t feasible_mask16(uint4 r)
{
    uint32_t w[4] = {r.x, r.y, r.z, r.w};
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 4; i++) {
        uint32_t x = w[i] & 0x7F7F7F7Fu;
#pragma unroll
        for (int b = 0; b < 4; b++)
            if (((x >> (8 * b)) & 0xFFu) == 0) m |= 1u << (4 * i + b);
    }
    return m;
}

// Visit the eligible candidates of one group of 16 (reason bytes r, first element e) in ascending order:
// f(rel, score_bits).
template <typename F>
__device__ __forceinline__ void for_each_eligible16(const DevPlan &P, const int32_t *vals, const SelArgs &A,
                                                    const uint8_t *cls, uint64_t e, const uint4 r, F f)
{
    // any byte with its low 7 bits clear?  (zero-byte test on the masked words; most groups have none)
    const uint32_t x0 = r.x & 0x7F7F7F7Fu, x1 = r.y & 0x7F7F7F7Fu, x2 = r.z & 0x7F7F7F7Fu, x3 = r.w & 0x7F7F7F7Fu;
    const uint32_t z = ((x0 - 0x01010101u) & ~x0) | ((x1 - 0x01010101u) & ~x1) | ((x2 - 0x01010101u) & ~x2) |
                       ((x3 - 0x01010101u) & ~x3);
    if ((z & 0x80808080u) == 0) return;
    uint32_t m = feasible_mask16(r);
    if (cls) {
        // bytes of a slab that is still being filled are not results yet: keep the candidates of evaluated slabs
        // (class byte 0) only.  The sixteen candidates lie in one slab or straddle one boundary.
        const uint64_t abs0 = A.first + e, s0 = abs0 / A.guard.slab;
        const uint32_t in0 = (uint32_t)min((uint64_t)16, (s0 + 1) * A.guard.slab - abs0);   // candidates in slab s0
        const uint64_t rel_s = s0 - A.guard.slab_lo;
        if (cls[rel_s] != 0) m &= ~((1u << in0) - 1u);
        if (in0 < 16u && (m >> in0) != 0u && rel_s + 1 < A.guard.n_slabs && cls[rel_s + 1] != 0) m &= (1u << in0) - 1u;
    }
    while (m) {
        int i = __ffs(m) - 1;
        m &= m - 1;
        uint64_t rel = e + i;
        if (in_sim_domain(P, vals, A.first + rel)) f(rel, __float_as_uint(__ldg(A.tput + rel)));
    }
}

constexpr int kSelTiles = 4;                               // tiles of 256 x 16 candidates per block
constexpr uint64_t kSelTile = (uint64_t)kSelThreads * 16;  // candidates per tile

// Load this thread's group of every tile of the block's chunk before any of them is looked at, so the
// reads of a chunk are all in flight together.
__device__ __forceinline__ void load_chunk(const SelArgs &A, uint64_t lo, uint64_t hi, uint4 (&r)[kSelTiles])
{
#pragma unroll
    for (int t = 0; t < kSelTiles; t++) {
        const uint64_t e = lo + (uint64_t)t * kSelTile + (uint64_t)threadIdx.x * 16;
        r[t] = e < hi ? load_reason16(A.reason, e, A.count) : make_uint4(~0u, ~0u, ~0u, ~0u);
    }
}

// One chunk of the histogram passes.  pass 0: every chunk; pass 1: the chunks on the eligible list.
__device__ __forceinline__ void sel_hist_chunk(const DevPlan &P, const SelArgs &A, const int32_t *vals, int pass,
                                               unsigned int chunk, unsigned int *s_elig)
{
    const uint64_t lo = (uint64_t)chunk * A.chunk;
    const uint64_t hi = min(lo + A.chunk, A.count);
    const uint8_t *cls = sel_guard_cls(A);
    if (pass == 0) {
        if (threadIdx.x == 0) *s_elig = 0;
        __syncthreads();
    }
    const uint32_t b1 = pass == 1 ? A.ctrl->b1 : 0;
    unsigned int mine = 0;
    uint4 r[kSelTiles];
    load_chunk(A, lo, hi, r);
#pragma unroll
    for (int t = 0; t < kSelTiles; t++) {
        const uint64_t e = lo + (uint64_t)t * kSelTile + (uint64_t)threadIdx.x * 16;
        for_each_eligible16(P, vals, A, cls, e, r[t], [&](uint64_t, uint32_t bits) {
            if (pass == 0) {
                atomicAdd(A.hist1 + (bits >> 16), 1u);
                atomicAdd(A.coarse1 + (bits >> 24), 1u);
                mine++;
            } else if ((bits >> 16) == b1) {
                atomicAdd(A.hist2 + (bits & 0xFFFFu), 1u);
                atomicAdd(A.coarse2 + ((bits >> 8) & 0xFFu), 1u);
            }
        });
    }
    if (pass == 0) {
        if (mine) atomicAdd(s_elig, mine);
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned int n = *s_elig;
            A.blk_elig[chunk] = n;
            // later passes only visit the chunks on this list
            if (n) A.elig_list[atomicAdd(&A.ctrl->n_elig, 1u)] = chunk;
        }
    }
}

__global__ void __launch_bounds__(kSelThreads) sel_hist_kernel(const __grid_constant__ DevPlan P, const SelArgs A,
                                                                const int32_t *vals, int pass)
{
    chain_enter();
    __shared__ unsigned int s_elig;
    if (pass == 0) {   // one block per chunk: the whole array is read, the more loads in flight the better
        sel_hist_chunk(P, A, vals, 0, blockIdx.x, &s_elig);
        return;
    }
    if (A.ctrl->take_all) return;   // nothing to refine
    const unsigned int n_list = A.ctrl->n_elig;
    const unsigned int n_chunks = (unsigned int)((A.count + A.chunk - 1) / A.chunk);
    (void)n_chunks;
    for (unsigned int li = blockIdx.x; li < n_list; li += gridDim.x)
        sel_hist_chunk(P, A, vals, 1, (unsigned int)PF_AT(P.chk, A.elig_list[li], n_chunks, PF_SITE_CHUNK), &s_elig);
}

// Block-wide inclusive prefix sum over 1024 threads (warp shuffles, then the warp totals).
__device__ __forceinline__ unsigned long long block_prefix_1024(unsigned long long x, unsigned long long *s_warp)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, off);
        if (lane >= off) x += y;
    }
    if (lane == 31) s_warp[warp] = x;
    __syncthreads();
    if (warp == 0) {
        unsigned long long t = s_warp[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, t, off);
            if (lane >= off) t += y;
        }
        s_warp[lane] = t;
    }
    __syncthreads();
    if (warp > 0) x += s_warp[warp - 1];
    __syncthreads();
    return x;
}

// One block of 256 threads: find the bin (scanning from the top) where the running count reaches the target.
// The coarse histogram (one entry per 256 fine bins) locates the group, the group's 256 fine bins the bin.
__device__ __forceinline__ unsigned long long block_prefix_256(unsigned long long x, unsigned long long *s_warp)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, off);
        if (lane >= off) x += y;
    }
    if (lane == 31) s_warp[warp] = x;
    __syncthreads();
    unsigned long long add = 0;
    for (int w = 0; w < warp; w++) add += s_warp[w];
    __syncthreads();
    return x + add;
}

__global__ void __launch_bounds__(256) sel_scan_kernel(const SelArgs A, int pass)
{
    chain_enter();
    __shared__ unsigned long long s_warp[8];
    __shared__ unsigned long long s_total, s_above;
    __shared__ int s_group;
    const int tid = threadIdx.x;
    SelCtrl *c = A.ctrl;
    if (pass == 1 && c->take_all) return;
    const unsigned int *fine = pass == 0 ? A.hist1 : A.hist2;
    const unsigned int *coarse = pass == 0 ? A.coarse1 : A.coarse2;
    // thread t owns coarse group 255 - t: an inclusive prefix over threads counts from the top
    const unsigned long long mine = coarse[255 - tid];
    const unsigned long long incl = block_prefix_256(mine, s_warp);
    if (tid == 255) s_total = incl;
    __syncthreads();
    const unsigned long long total = s_total;
    unsigned long long target;
    if (pass == 0) {
        target = A.s_max;
        if (tid == 0) {
            c->total = total;
            c->target = target;
            c->take_all = total <= target ? 1 : 0;
            if (total <= target) {
                c->thr_bits = 0;
                c->n_gt = total;
                c->need_eq = 0;
            }
        }
        if (total <= target) return;
    } else {
        target = c->target - c->above1;
    }
    if (incl - mine < target && incl >= target) {
        s_group = 255 - tid;
        s_above = incl - mine;
    }
    __syncthreads();
    // same search inside the group's 256 fine bins
    const int g = s_group;
    const unsigned long long fm = fine[g * 256 + (255 - tid)];
    const unsigned long long fincl = s_above + block_prefix_256(fm, s_warp);
    if (fincl - fm < target && fincl >= target) {
        const uint32_t bin = (uint32_t)(g * 256 + (255 - tid));
        const unsigned long long run = fincl - fm;   // eligible strictly above this bin
        if (pass == 0) {
            c->b1 = bin;
            c->above1 = run;
        } else {
            c->thr_bits = (c->b1 << 16) | bin;
            c->n_gt = c->above1 + run;
            c->need_eq = c->target - (c->above1 + run);
        }
    }
}

// Per-chunk counts of admitted candidates, for the chunks on the eligible list (the others keep their zeros).
__global__ void __launch_bounds__(kSelThreads) sel_count_kernel(const __grid_constant__ DevPlan P, const SelArgs A,
                                                                 const int32_t *vals)
{
    chain_enter();
    __shared__ unsigned int s_gt, s_eq;
    const unsigned int n_list = A.ctrl->n_elig;
    const bool all = A.ctrl->take_all != 0;
    const uint32_t thr = A.ctrl->thr_bits;
    const uint8_t *cls = sel_guard_cls(A);
    for (unsigned int li = blockIdx.x; li < n_list; li += gridDim.x) {
        const unsigned int chunk = (unsigned int)PF_AT(P.chk, A.elig_list[li], (A.count + A.chunk - 1) / A.chunk, PF_SITE_CHUNK);
        if (all) {   // every eligible candidate is taken: the first pass has counted them already
            if (threadIdx.x == 0) {
                A.blk_gt[chunk] = A.blk_elig[chunk];
                A.blk_eq[chunk] = 0;
            }
            continue;
        }
        if (threadIdx.x == 0) s_gt = s_eq = 0;
        __syncthreads();
        const uint64_t lo = (uint64_t)chunk * A.chunk;
        const uint64_t hi = min(lo + A.chunk, A.count);
        unsigned int gt = 0, eq = 0;
        uint4 r[kSelTiles];
        load_chunk(A, lo, hi, r);
#pragma unroll
        for (int t = 0; t < kSelTiles; t++) {
            const uint64_t e = lo + (uint64_t)t * kSelTile + (uint64_t)threadIdx.x * 16;
            for_each_eligible16(P, vals, A, cls, e, r[t], [&](uint64_t, uint32_t bits) {
                if (bits > thr) gt++;
                else if (bits == thr) eq++;
            });
        }
        if (gt) atomicAdd(&s_gt, gt);
        if (eq) atomicAdd(&s_eq, eq);
        __syncthreads();
        if (threadIdx.x == 0) {
            A.blk_gt[chunk] = s_gt;
            A.blk_eq[chunk] = s_eq;
        }
        __syncthreads();
    }
}

// Exclusive prefix over the per-chunk counts + the survivor count.  One block; both counts travel through one
// scan as (greater << 32 | equal) -- their totals stay below 2^32.  Up to kScanTiles * 1024 chunks are scanned
// in one go: every thread holds one entry of every tile, the tiles' warp-level scans run side by side, and one
// round through shared memory turns the warp totals into offsets.  Longer lists are walked tile by tile.
constexpr int kScanTiles = 16;
__global__ void __launch_bounds__(1024) sel_blockscan_kernel(const SelArgs A, int nblocks)
{
    chain_enter();
    __shared__ unsigned long long s_warp[32];
    __shared__ unsigned long long s_tot[kScanTiles][33];   // warp totals per tile, then their exclusive prefixes
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long grand = 0ull;   // totals over all chunks: greater << 32 | equal
    if (nblocks <= kScanTiles * 1024) {
        const int tiles = (nblocks + 1023) / 1024;
        unsigned long long v[kScanTiles], x[kScanTiles];
#pragma unroll
        for (int k = 0; k < kScanTiles; k++) {
            const int b = k * 1024 + tid;
            v[k] = (k < tiles && b < nblocks) ? ((A.blk_gt[b] << 32) | A.blk_eq[b]) : 0ull;
            x[k] = v[k];
        }
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
#pragma unroll
            for (int k = 0; k < kScanTiles; k++) {
                const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x[k], off);
                if (lane >= off) x[k] += y;
            }
        }
        if (lane == 31) {
#pragma unroll
            for (int k = 0; k < kScanTiles; k++) s_tot[k][warp] = x[k];
        }
        __syncthreads();
        // warp k turns tile k's 32 warp totals into exclusive prefixes and leaves the tile total in slot 32
        if (warp < kScanTiles) {
            const unsigned long long t = s_tot[warp][lane];
            unsigned long long incl = t;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += y;
            }
            s_tot[warp][lane] = incl - t;
            if (lane == 31) s_tot[warp][32] = incl;
        }
        __syncthreads();
        unsigned long long carry = 0ull;
#pragma unroll
        for (int k = 0; k < kScanTiles; k++) {
            const int b = k * 1024 + tid;
            if (k < tiles && b < nblocks) {
                const unsigned long long excl = carry + s_tot[k][warp] + x[k] - v[k];
                A.blk_gt[b] = excl >> 32;
                A.blk_eq[b] = excl & 0xFFFFFFFFull;
            }
            carry += s_tot[k][32];
        }
        grand = carry;
    } else {
        unsigned long long carry = 0ull;
        unsigned long long nxt = tid < nblocks ? ((A.blk_gt[tid] << 32) | A.blk_eq[tid]) : 0ull;
        for (int base = 0; base < nblocks; base += 1024) {
            const int b = base + tid, bn = b + 1024;
            const unsigned long long cur = nxt;
            nxt = bn < nblocks ? ((A.blk_gt[bn] << 32) | A.blk_eq[bn]) : 0ull;
            const unsigned long long incl = block_prefix_1024(cur, s_warp);
            const unsigned long long total = s_warp[31];
            const unsigned long long excl = carry + incl - cur;
            if (b < nblocks) {
                A.blk_gt[b] = excl >> 32;
                A.blk_eq[b] = excl & 0xFFFFFFFFull;
            }
            carry += total;
            __syncthreads();   // s_warp is rewritten by the next tile's scan
        }
        grand = carry;
    }
    if (tid == 0) {
        // taken here: everything above the threshold, and of those at it what the cut leaves for this range
        const SelCtrl *c = A.ctrl;
        const unsigned long long need = (c->take_all || c->need_eq <= A.eq_before) ? 0ull : c->need_eq - A.eq_before;
        const unsigned long long n_eq = grand & 0xFFFFFFFFull;
        *A.surv_count = (grand >> 32) + (n_eq < need ? n_eq : need);
    }
}

// Ordered write: position of an admitted candidate = (# taken "greater" before it) + min(# "equal" before it, need_eq)
__device__ __forceinline__ void sel_write_chunk(const DevPlan &P, const SelArgs &A, const int32_t *vals,
                                                unsigned int chunk, unsigned int *s_gt,
                                                unsigned long long &s_run_gt, unsigned long long &s_run_eq)
{
    const int tid = threadIdx.x;
    const uint64_t lo = (uint64_t)chunk * A.chunk;
    const uint64_t hi = min(lo + A.chunk, A.count);
    const uint32_t thr = A.ctrl->thr_bits;
    const bool all = A.ctrl->take_all != 0;
    const unsigned long long need_eq =
        (all || A.ctrl->need_eq <= A.eq_before) ? 0ull : A.ctrl->need_eq - A.eq_before;
    const uint8_t *cls = sel_guard_cls(A);
    if (tid == 0) {
        s_run_gt = A.blk_gt[chunk];
        s_run_eq = A.blk_eq[chunk];
    }
    uint4 r[kSelTiles];
    load_chunk(A, lo, hi, r);
    __syncthreads();
#pragma unroll
    for (int t = 0; t < kSelTiles; t++) {
        const uint64_t e = lo + (uint64_t)t * kSelTile + (uint64_t)tid * 16;
        unsigned int gt = 0, eq = 0;
        for_each_eligible16(P, vals, A, cls, e, r[t], [&](uint64_t, uint32_t bits) {
            if (all || bits > thr) gt++;
            else if (bits == thr) eq++;
        });
        if (!__syncthreads_or((int)(gt | eq))) continue;   // nothing eligible in this tile (the common case)
        // inclusive scan of the per-thread counts: both travel as (gt << 16 | eq) -- a thread holds at most 16 of
        // each, a tile at most 4096 -- through warp shuffles, then across the eight warp totals
        const int lane = tid & 31, warp = tid >> 5;
        unsigned int x = (gt << 16) | eq;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned int y = __shfl_up_sync(0xFFFFFFFFu, x, off);
            if (lane >= off) x += y;
        }
        if (lane == 31) s_gt[warp] = x;
        __syncthreads();
        unsigned int before = 0, total = 0;
#pragma unroll
        for (int w = 0; w < kSelThreads / 32; w++) {
            const unsigned int wt = s_gt[w];
            if (w < warp) before += wt;
            total += wt;
        }
        x += before;
        unsigned long long my_gt = s_run_gt + ((x >> 16) - gt);
        unsigned long long my_eq = s_run_eq + ((x & 0xFFFFu) - eq);
        if (gt | eq)
            for_each_eligible16(P, vals, A, cls, e, r[t], [&](uint64_t rel, uint32_t bits) {
                if (all || bits > thr) {
                    unsigned long long pos = my_gt + (my_eq < need_eq ? my_eq : need_eq);
                    (void)PF_AT(P.chk, pos, A.s_max, PF_SITE_SURVIVOR);
                    if (pos < A.s_max) A.surv_idx[pos] = A.first + rel;   // s_max: the list's capacity
                    my_gt++;
                } else if (bits == thr) {
                    if (my_eq < need_eq && my_gt + my_eq < A.s_max) A.surv_idx[my_gt + my_eq] = A.first + rel;
                    my_eq++;
                }
            });
        __syncthreads();
        if (tid == 0) {
            s_run_gt += total >> 16;
            s_run_eq += total & 0xFFFFu;
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kSelThreads) sel_write_kernel(const __grid_constant__ DevPlan P, const SelArgs A,
                                                                 const int32_t *vals)
{
    chain_enter();
    __shared__ unsigned int s_gt[kSelThreads / 32];   // warp totals of a tile's scan
    __shared__ unsigned long long s_run_gt, s_run_eq;
    const unsigned int n_list = A.ctrl->n_elig;
    for (unsigned int li = blockIdx.x; li < n_list; li += gridDim.x) {
        sel_write_chunk(P, A, vals, (unsigned int)PF_AT(P.chk, A.elig_list[li], (A.count + A.chunk - 1) / A.chunk, PF_SITE_CHUNK),
                        s_gt, s_run_gt, s_run_eq);
        __syncthreads();   // the running offsets are reset by the next chunk
    }
}

struct SelLayout {
    size_t off_ctrl, off_hist1, off_hist2, off_coarse, off_gt, off_eq, off_elig, off_list, total;
    int nblocks;
    uint64_t chunk;
};

static SelLayout sel_layout(const pf_plan_t *p, uint64_t count)
{
    SelLayout l;
    // contiguous chunks of kSelTiles tiles (256 threads x 16 candidates each): many more blocks than SMs, so a
    // chunk that happens to hold most of the feasible candidates does not hold up the rest
    uint64_t chunk = (uint64_t)kSelTiles * kSelTile;
    l.chunk = chunk;
    l.nblocks = (int)((count + chunk - 1) / chunk);
    if (l.nblocks < 1) l.nblocks = 1;
    l.off_ctrl = 0;
    l.off_hist1 = 256;
    l.off_hist2 = l.off_hist1 + kBins * 4;
    l.off_coarse = l.off_hist2 + kBins * 4;          // coarse1[256], coarse2[256]
    l.off_gt = l.off_coarse + 2 * 256 * 4;
    size_t per = (((size_t)l.nblocks + 1) * 8 + 255) & ~(size_t)255;
    l.off_eq = l.off_gt + per;
    l.off_elig = l.off_eq + per;
    l.off_list = l.off_elig + per;
    l.total = l.off_list + per;
    return l;
}

}  // namespace pf

using namespace pf;

extern "C" size_t pf_select_workspace(const pf_plan_t *p, uint64_t count, uint64_t s_max)
{
    (void)s_max;
    if (!p) return 0;
    return sel_layout(p, count).total;
}

extern "C" int pf_select_survivors(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason,
                                   const float *d_tput, uint64_t s_max, uint64_t *d_surv_idx, uint64_t *d_surv_count,
                                   void *d_workspace, size_t workspace_bytes, void *stream)
{
    return select_run(p, first, count, d_reason, d_tput, s_max, d_surv_idx, d_surv_count, d_workspace,
                      workspace_bytes, (cudaStream_t)stream, false, nullptr);
}

// Zero the selection's control words, histograms and per-chunk counts and say where the scoring kernel may collect
// the first pass's results (the fused search call: clear -> score with digest -> select_run(have_digest)).
int pf::select_clear(pf_plan_t *p, uint64_t count, void *d_workspace, size_t workspace_bytes, cudaStream_t st,
                     ScoreDigest *dg_out)
{
    if (!p || count == 0 || count >= PF_MAX_COUNT) return PF_ERANGE;
    const SelLayout lay = sel_layout(p, count);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < lay.total) return PF_EWORKSPACE;
    uint8_t *ws = (uint8_t *)d_workspace;
    PF_CUDA_TRY(cudaMemsetAsync(ws, 0, lay.off_list, st), "selection workspace: clear");
    if (dg_out) {
        dg_out->hist1 = (unsigned int *)(ws + lay.off_hist1);
        dg_out->coarse1 = (unsigned int *)(ws + lay.off_coarse);
        dg_out->elig = (unsigned int *)(ws + lay.off_elig);
        dg_out->list = (unsigned int *)(ws + lay.off_list);
        dg_out->n_list = &((SelCtrl *)(ws + lay.off_ctrl))->n_elig;
        dg_out->chunk = (uint32_t)lay.chunk;
    }
    return PF_OK;
}

int pf::select_run(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
                   uint64_t s_max, uint64_t *d_surv_idx, uint64_t *d_surv_count, void *d_workspace,
                   size_t workspace_bytes, cudaStream_t st, bool have_digest, const FillGuard *guard)
{
    if (!p || !d_reason || !d_tput || !d_surv_idx || !d_surv_count) return PF_EINVAL;
    if (p->dev.phase != PF_PHASE_TRAIN) return PF_EUNSUPPORTED;
    if (count == 0 || count >= PF_MAX_COUNT || s_max == 0) return PF_ERANGE;
    if (first >= p->size || count > p->size - first) return PF_ERANGE;
    const SelLayout lay = sel_layout(p, count);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < lay.total) return PF_EWORKSPACE;
    if (int rc_dev = check_device(p)) return rc_dev;
    uint8_t *ws = (uint8_t *)d_workspace;
    SelArgs a;
    a.first = first; a.count = count; a.s_max = s_max; a.reason = d_reason; a.tput = d_tput;
    a.ctrl = (SelCtrl *)(ws + lay.off_ctrl);
    a.hist1 = (unsigned int *)(ws + lay.off_hist1);
    a.hist2 = (unsigned int *)(ws + lay.off_hist2);
    a.coarse1 = (unsigned int *)(ws + lay.off_coarse);
    a.coarse2 = a.coarse1 + 256;
    a.blk_elig = (unsigned int *)(ws + lay.off_elig);
    a.elig_list = (unsigned int *)(ws + lay.off_list);
    a.blk_gt = (unsigned long long *)(ws + lay.off_gt);
    a.blk_eq = (unsigned long long *)(ws + lay.off_eq);
    a.surv_idx = d_surv_idx; a.surv_count = d_surv_count; a.chunk = lay.chunk;
    a.eq_before = 0ull;
    if (guard) a.guard = *guard;
    // control words, histograms and the per-chunk counts start at zero (chunks that are not on the eligible list
    // are never written again); with a digest the scoring kernel has filled the first pass's part already
    if (!have_digest) PF_CUDA_TRY(cudaMemsetAsync(ws, 0, lay.off_elig, st), "pf_select_survivors: clear");
    // the passes after the first visit the eligible chunks only: a grid that fills the GPU walks the list
    const int list_grid = lay.nblocks < p->sm_count * 8 ? lay.nblocks : p->sm_count * 8;
    timing_begin(p, PF_T_SELECT, st);
    int launches = 6;
    if (!have_digest) {
        sel_hist_kernel<<<lay.nblocks, kSelThreads, 0, st>>>(p->dev, a, p->d_vals, 0);
        launches++;
    }
    sel_scan_kernel<<<1, 256, 0, st>>>(a, 0);
    launch_chained(sel_hist_kernel, list_grid, kSelThreads, 0, st, p->dev, a, p->d_vals, 1);
    launch_chained(sel_scan_kernel, 1, 256, 0, st, a, 1);
    launch_chained(sel_count_kernel, list_grid, kSelThreads, 0, st, p->dev, a, p->d_vals);
    launch_chained(sel_blockscan_kernel, 1, 1024, 0, st, a, lay.nblocks);
    launch_chained(sel_write_kernel, list_grid, kSelThreads, 0, st, p->dev, a, p->d_vals);
    timing_end(p, PF_T_SELECT, launches, st);
    for (int i = 0; i < launches; i++) count_launch();
    PF_CUDA_TRY(cudaGetLastError(), "pf_select_survivors launch");
    return PF_OK;
}

// ------------------------------------------------------------------ the selection in steps, for one space split
// over several GPUs: every rank histograms its own slice, the histograms are summed by the caller, the cut is
// found on the sums, every rank compacts its slice against the same cut.

namespace pf {

// One block: scanning a 65,536-bin histogram of 64-bit counts from the top bin down, find the bin in which the
// running count reaches `target`.  Thread t owns the 64 bins just below 65536 - 64 t.
__global__ void __launch_bounds__(1024) sel_cut_kernel(const unsigned long long *hist, int level, uint64_t s_max,
                                                       SelCtrl *c)
{
    __shared__ unsigned long long s_warp[32];
    const int tid = threadIdx.x;
    if (level == 1 && c->take_all) return;
    const int top = kBins - 1 - 64 * tid;   // this thread's highest bin
    unsigned long long mine = 0ull;
    for (int j = 0; j < 64; j++) mine += hist[top - j];
    const unsigned long long incl = block_prefix_1024(mine, s_warp);
    __shared__ unsigned long long s_total;
    if (tid == 1023) s_total = incl;
    __syncthreads();
    unsigned long long target;
    if (level == 0) {
        const unsigned long long total = s_total;
        target = s_max;
        if (tid == 0) {
            c->total = total;
            c->target = target;
            c->take_all = total <= target ? 1 : 0;
            c->n_elig = 0;
            if (total <= target) {
                c->b1 = 0;
                c->above1 = 0;
                c->thr_bits = 0;
                c->n_gt = total;
                c->need_eq = 0;
            }
        }
        if (total <= target) return;
    } else {
        target = c->target - c->above1;
    }
    if (incl - mine < target && incl >= target) {
        unsigned long long run = incl - mine;   // count strictly above the bin under test
        for (int j = 0; j < 64; j++) {
            const unsigned long long h = hist[top - j];
            if (run + h >= target) {
                const uint32_t bin = (uint32_t)(top - j);
                if (level == 0) {
                    c->b1 = bin;
                    c->above1 = run;
                } else {
                    c->thr_bits = (c->b1 << 16) | bin;
                    c->n_gt = c->above1 + run;
                    c->need_eq = c->target - (c->above1 + run);
                }
                break;
            }
            run += h;
        }
    }
}

static int sel_args(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
                    void *d_workspace, size_t workspace_bytes, SelArgs &a, SelLayout &lay)
{
    if (!p || !d_reason || !d_tput) return PF_EINVAL;
    if (p->dev.phase != PF_PHASE_TRAIN) return PF_EUNSUPPORTED;
    if (count == 0 || count >= PF_MAX_COUNT) return PF_ERANGE;
    if (first >= p->size || count > p->size - first) return PF_ERANGE;
    lay = sel_layout(p, count);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < lay.total) return PF_EWORKSPACE;
    if (int rc_dev = check_device(p)) return rc_dev;
    uint8_t *ws = (uint8_t *)d_workspace;
    a.first = first; a.count = count; a.s_max = 0; a.reason = d_reason; a.tput = d_tput;
    a.ctrl = (SelCtrl *)(ws + lay.off_ctrl);
    a.hist1 = (unsigned int *)(ws + lay.off_hist1);
    a.hist2 = (unsigned int *)(ws + lay.off_hist2);
    a.coarse1 = (unsigned int *)(ws + lay.off_coarse);
    a.coarse2 = a.coarse1 + 256;
    a.blk_elig = (unsigned int *)(ws + lay.off_elig);
    a.elig_list = (unsigned int *)(ws + lay.off_list);
    a.blk_gt = (unsigned long long *)(ws + lay.off_gt);
    a.blk_eq = (unsigned long long *)(ws + lay.off_eq);
    a.surv_idx = nullptr; a.surv_count = nullptr; a.chunk = lay.chunk;
    a.eq_before = 0ull;
    return PF_OK;
}

}  // namespace pf

extern "C" int pf_select_hist(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason,
                              const float *d_tput, const pf_select_cut_t *d_cut, uint32_t *d_hist, void *d_workspace,
                              size_t workspace_bytes, void *stream)
{
    if (!d_hist) return PF_EINVAL;
    SelArgs a;
    SelLayout lay;
    int rc = sel_args(p, first, count, d_reason, d_tput, d_workspace, workspace_bytes, a, lay);
    if (rc != PF_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)d_workspace;
    PF_CUDA_TRY(cudaMemsetAsync(ws, 0, lay.off_list, st), "pf_select_hist: clear");
    PF_CUDA_TRY(cudaMemsetAsync(d_hist, 0, kBins * sizeof(uint32_t), st), "pf_select_hist: clear");
    timing_begin(p, PF_T_SELECT, st);
    int launches = 1;
    if (!d_cut) {
        a.hist1 = d_hist;                     // level 0: the high 16 score bits of every eligible candidate
        sel_hist_kernel<<<lay.nblocks, kSelThreads, 0, st>>>(p->dev, a, p->d_vals, 0);
    } else {
        // level 1: the low 16 bits of those whose high bits are the cut's bin.  The chunk list comes from a
        // level-0 pass into scratch; the cut's fields are copied behind it (the list length survives).
        sel_hist_kernel<<<lay.nblocks, kSelThreads, 0, st>>>(p->dev, a, p->d_vals, 0);
        PF_CUDA_TRY(cudaMemcpyAsync(a.ctrl, d_cut, offsetof(SelCtrl, n_elig), cudaMemcpyDeviceToDevice, st),
                    "pf_select_hist: cut");
        a.hist2 = d_hist;
        const int list_grid = lay.nblocks < p->sm_count * 8 ? lay.nblocks : p->sm_count * 8;
        sel_hist_kernel<<<list_grid, kSelThreads, 0, st>>>(p->dev, a, p->d_vals, 1);
        launches = 2;
    }
    timing_end(p, PF_T_SELECT, launches, st);
    for (int i = 0; i < launches; i++) count_launch();
    PF_CUDA_TRY(cudaGetLastError(), "pf_select_hist launch");
    return PF_OK;
}

extern "C" int pf_select_cut(const uint64_t *d_hist, int level, uint64_t s_max, pf_select_cut_t *d_cut, void *stream)
{
    if (!d_hist || !d_cut || (level != 0 && level != 1)) return PF_EINVAL;
    if (level == 0 && s_max == 0) return PF_ERANGE;
    sel_cut_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>((const unsigned long long *)d_hist, level, s_max,
                                                         (SelCtrl *)d_cut);
    count_launch();
    PF_CUDA_TRY(cudaGetLastError(), "pf_select_cut launch");
    return PF_OK;
}

extern "C" int pf_select_write(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason,
                               const float *d_tput, const pf_select_cut_t *d_cut, uint64_t eq_before,
                               uint64_t *d_surv_idx, uint64_t surv_cap, uint64_t *d_surv_count, void *d_workspace,
                               size_t workspace_bytes, void *stream)
{
    if (!d_cut || !d_surv_idx || !d_surv_count) return PF_EINVAL;
    SelArgs a;
    SelLayout lay;
    int rc = sel_args(p, first, count, d_reason, d_tput, d_workspace, workspace_bytes, a, lay);
    if (rc != PF_OK) return rc;
    if (surv_cap == 0) return PF_ERANGE;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = (uint8_t *)d_workspace;
    a.surv_idx = d_surv_idx; a.surv_count = d_surv_count; a.eq_before = eq_before;
    a.s_max = surv_cap;   // entries past the capacity are counted but not written
    PF_CUDA_TRY(cudaMemsetAsync(ws, 0, lay.off_list, st), "pf_select_write: clear");
    timing_begin(p, PF_T_SELECT, st);
    // the chunk list and per-chunk eligible counts (a level-0 pass into scratch), then the cut, then the usual
    // count / prefix / ordered write
    sel_hist_kernel<<<lay.nblocks, kSelThreads, 0, st>>>(p->dev, a, p->d_vals, 0);
    PF_CUDA_TRY(cudaMemcpyAsync(a.ctrl, d_cut, offsetof(SelCtrl, n_elig), cudaMemcpyDeviceToDevice, st),
                "pf_select_write: cut");
    const int list_grid = lay.nblocks < p->sm_count * 8 ? lay.nblocks : p->sm_count * 8;
    sel_count_kernel<<<list_grid, kSelThreads, 0, st>>>(p->dev, a, p->d_vals);
    sel_blockscan_kernel<<<1, 1024, 0, st>>>(a, lay.nblocks);
    sel_write_kernel<<<list_grid, kSelThreads, 0, st>>>(p->dev, a, p->d_vals);
    timing_end(p, PF_T_SELECT, 4, st);
    for (int i = 0; i < 4; i++) count_launch();
    PF_CUDA_TRY(cudaGetLastError(), "pf_select_write launch");
    return PF_OK;
}
