// pf_compact.cu -- a compact view of a scoring call's dense outputs: how many candidates each rule rejected, one
// feasibility bit per candidate, and the feasible plans as packed records in ascending index order.  In the spaces
// this library is built for a few candidates in ten thousand are feasible, so a caller that wants "which plans pass,
// with what score and memory, and why the others fail" can take this view across a host link instead of thirteen
// bytes per candidate.
//
// Three launches: per chunk of 16,384 candidates, the reason histogram (in shared memory, one column per thread),
// the feasibility bits and the chunk's feasible count; one block's exclusive prefix over the chunk counts; the
// ordered write of the records, which only the chunks that hold a feasible plan take part in.
#include "pf_internal.cuh"

namespace pf {

constexpr int kCmpThreads = 256;
constexpr int kCmpTiles = 4;                                  // tiles of 256 x 16 candidates per block
constexpr uint64_t kCmpTile = (uint64_t)kCmpThreads * 16;
constexpr uint64_t kCmpChunk = kCmpTiles * kCmpTile;
constexpr int kCmpBins = 16;                                  // reason codes 0..11 (the rest stay empty)

struct CompactArgs {
    uint64_t first, count;
    const uint8_t *reason;
    const float *tput;
    const long long *mem;            // may be NULL
    unsigned long long *hist;        // [kCmpBins], zeroed by the host
    uint8_t *mask;                   // may be NULL; ceil(count / 8) bytes, bit i of byte i / 8 = candidate first + i
    pf_record_t *records;            // may be NULL
    uint64_t record_cap;
    unsigned long long *n_feasible;
    unsigned int *chunk_count;       // [n_chunks] feasible per chunk, then exclusive prefixes (as 64-bit pairs below)
    unsigned long long *chunk_pre;   // [n_chunks]
    unsigned int n_chunks;
    FillGuard guard;                 // cls != NULL: constant blocks may still be in flight; take their bytes from the classes
};

// class bytes to consult, or NULL when every block of the dense outputs may be read
__device__ __forceinline__ const uint8_t *cmp_guard_cls(const CompactArgs &A)
{
    const FillGuard &g = A.guard;
    if (!g.cls || !order_table_valid(g.hdr, g.slab_lo, g.n_slabs, g.tail, g.fpe)) return nullptr;
    return g.cls;
}

// 16 reason bytes starting at candidate e of the range (bytes past the end read as 0xFF = not a candidate)
__device__ __forceinline__ uint4 cmp_load16(const uint8_t *reason, uint64_t e, uint64_t count)
{
    if (e + 16 <= count && (((uintptr_t)(reason + e)) & 15) == 0) return __ldg(reinterpret_cast<const uint4 *>(reason + e));
    uint32_t w[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
    for (int i = 0; i < 16; i++)
        if (e + i < count) {
            const uint32_t b = reason[e + i];
            w[i >> 2] = (w[i >> 2] & ~(0xFFu << (8 * (i & 3)))) | (b << (8 * (i & 3)));
        }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// The 16 reason bytes of candidates [e, e + 16) of the range.  With class bytes (cls), the bytes of candidates in a
// constant block are the block's class -- what the streaming kernel writes there, sooner or later -- and memory is
// read only where an evaluated block is involved.
__device__ __forceinline__ uint4 cmp_reason16(const CompactArgs &A, const uint8_t *cls, uint64_t e)
{
    if (!cls) return cmp_load16(A.reason, e, A.count);
    const FillGuard &g = A.guard;
    const uint64_t a0 = A.first + e;
    const uint64_t last = (e + 15 < A.count ? e + 15 : A.count - 1) + A.first;
    const uint64_t s0 = a0 / g.slab - g.slab_lo, s1 = last / g.slab - g.slab_lo;
    const uint32_t c0 = s0 < g.n_slabs ? cls[s0] : 0u;
    if (s0 == s1) {
        if (c0 == 0u) return cmp_load16(A.reason, e, A.count);
        const uint32_t w = c0 * 0x01010101u;
        return make_uint4(w, w, w, w);
    }
    // the group straddles blocks (at most two when a block holds 16 candidates or more; any number otherwise)
    uint4 r = cmp_load16(A.reason, e, A.count);
    uint32_t w[4] = {r.x, r.y, r.z, r.w};
    for (int i = 0; i < 16; i++) {
        if (e + i >= A.count) break;
        const uint64_t si = (a0 + i) / g.slab - g.slab_lo;
        const uint32_t c = si < g.n_slabs ? cls[si] : 0u;
        if (c != 0u) w[i >> 2] = (w[i >> 2] & ~(0xFFu << (8 * (i & 3)))) | (c << (8 * (i & 3)));
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// bit i set: byte i of the 16 is a feasible candidate's reason ((b & 0x7f) == 0; 0xFF padding is not)
__device__ __forceinline__ uint32_t cmp_feasible16(uint4 r)
{
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const uint32_t x = w[i] & 0x7F7F7F7Fu;
        // the word-level test says whether any byte is zero (almost never); which ones is then tested byte by byte
        if ((((x - 0x01010101u) & ~x) & 0x80808080u) == 0u) continue;
#pragma unroll
        for (int b = 0; b < 4; b++)
            if (((x >> (8 * b)) & 0xFFu) == 0u) m |= 1u << (4 * i + b);
    }
    return m;
}

__global__ void __launch_bounds__(kCmpThreads) compact_count_kernel(const CompactArgs A)
{
    __shared__ unsigned int s_hist[kCmpBins][kCmpThreads];   // one column per thread: no atomics, no conflicts
    __shared__ unsigned int s_feas;
    const int tid = threadIdx.x;
#pragma unroll
    for (int b = 0; b < kCmpBins; b++) s_hist[b][tid] = 0u;
    if (tid == 0) s_feas = 0u;
    __syncthreads();
    const uint64_t lo = (uint64_t)blockIdx.x * kCmpChunk;
    const uint8_t *cls = cmp_guard_cls(A);
    if (cls) {
        // A chunk that lies in constant blocks only (most do) needs no look at its candidates: each block adds its
        // overlap with the chunk to its class's bin, the chunk's bits are zero and it holds no feasible plan.
        const FillGuard &g = A.guard;
        const uint64_t hi = lo + kCmpChunk < A.count ? lo + kCmpChunk : A.count;
        const uint64_t s_first = (A.first + lo) / g.slab - g.slab_lo, s_last = (A.first + hi - 1) / g.slab - g.slab_lo;
        bool constant = true;
        for (uint64_t sl = s_first + tid; sl <= s_last; sl += kCmpThreads) constant &= sl < g.n_slabs && cls[sl] != 0;
        if (__syncthreads_and(constant)) {
            for (uint64_t sl = s_first + tid; sl <= s_last; sl += kCmpThreads) {
                const uint64_t b0 = (g.slab_lo + sl) * (uint64_t)g.slab, b1 = b0 + g.slab;
                const uint64_t a0 = b0 > A.first + lo ? b0 : A.first + lo, a1 = b1 < A.first + hi ? b1 : A.first + hi;
                atomicAdd(A.hist + (cls[sl] & 0x7Fu & (kCmpBins - 1)), (unsigned long long)(a1 - a0));
            }
            if (A.mask) {
                // the chunk starts at a multiple of 8 candidates; its last byte may be partial (end of the range)
                const uint64_t m0 = lo >> 3, m1 = (hi + 7) >> 3;
                for (uint64_t i = m0 + tid; i < m1; i += kCmpThreads) A.mask[i] = 0;
            }
            if (tid == 0) A.chunk_count[blockIdx.x] = 0u;
            return;
        }
    }
    uint4 r[kCmpTiles];
#pragma unroll
    for (int t = 0; t < kCmpTiles; t++) {
        const uint64_t e = lo + (uint64_t)t * kCmpTile + (uint64_t)tid * 16;
        r[t] = e < A.count ? cmp_reason16(A, cls, e) : make_uint4(~0u, ~0u, ~0u, ~0u);
    }
    unsigned int feas = 0;
#pragma unroll
    for (int t = 0; t < kCmpTiles; t++) {
        const uint64_t e = lo + (uint64_t)t * kCmpTile + (uint64_t)tid * 16;
        if (e >= A.count) continue;
        const uint32_t w[4] = {r[t].x, r[t].y, r[t].z, r[t].w};
        const uint32_t b0 = w[0] & 0xFFu;
        if (w[0] == b0 * 0x01010101u && w[1] == w[0] && w[2] == w[0] && w[3] == w[0] && e + 16 <= A.count) {
            // sixteen equal bytes (inside a block of candidates that one rule rejects): one update
            s_hist[b0 & 0x7Fu & (kCmpBins - 1)][tid] += 16u;
            if ((b0 & 0x7Fu) == 0u) feas += 16u;
        } else {
#pragma unroll
            for (int i = 0; i < 16; i++)
                if (e + i < A.count) {
                    const uint32_t b = (w[i >> 2] >> (8 * (i & 3))) & 0x7Fu;
                    s_hist[b & (kCmpBins - 1)][tid] += 1u;
                    feas += b == 0u;
                }
        }
        if (A.mask) {
            const uint32_t m = cmp_feasible16(r[t]);
            // the thread's sixteen bits are two mask bytes; the range starts at a multiple of 16 candidates per
            // thread, so they never share a byte with a neighbour
            uint8_t *dst = A.mask + (e >> 3);
            dst[0] = (uint8_t)(m & 0xFFu);
            if (e + 8 < A.count) dst[1] = (uint8_t)(m >> 8);
        }
    }
    if (feas) atomicAdd(&s_feas, feas);
    __syncthreads();
    // column sums: thread b < 16 adds up row b
    if (tid < kCmpBins) {
        unsigned long long sum = 0;
        for (int i = 0; i < kCmpThreads; i++) sum += s_hist[tid][(i + tid) & (kCmpThreads - 1)];
        if (sum) atomicAdd(A.hist + tid, sum);
    }
    if (tid == 0) A.chunk_count[blockIdx.x] = s_feas;
}

// exclusive prefix over the chunk counts (one block walks them 1024 at a time) and the total
__global__ void __launch_bounds__(1024) compact_scan_kernel(const CompactArgs A)
{
    __shared__ unsigned long long s_warp[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long carry = 0ull;   // chunks before this tile; the same in every thread
    for (unsigned int base = 0; base < A.n_chunks; base += 1024) {
        const unsigned int c = base + tid;
        const unsigned long long v = c < A.n_chunks ? A.chunk_count[c] : 0ull;
        unsigned long long x = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, off);
            if (lane >= off) x += y;
        }
        if (lane == 31) s_warp[warp] = x;
        __syncthreads();
        if (warp == 0) {   // inclusive prefix of the warp totals
            unsigned long long t = s_warp[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, t, off);
                if (lane >= off) t += y;
            }
            s_warp[lane] = t;
        }
        __syncthreads();
        const unsigned long long warps_before = warp ? s_warp[warp - 1] : 0ull;
        if (c < A.n_chunks) A.chunk_pre[c] = carry + warps_before + x - v;
        carry += s_warp[31];
        __syncthreads();   // s_warp is rewritten by the next tile
    }
    if (tid == 0) *A.n_feasible = carry;
}

// ordered write: a chunk's records start at its prefix; inside the chunk, tiles in order, threads in order,
// candidates in order
__global__ void __launch_bounds__(kCmpThreads) compact_write_kernel(const CompactArgs A)
{
    __shared__ unsigned int s_warp[kCmpThreads / 32];
    __shared__ unsigned long long s_run;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint8_t *cls = cmp_guard_cls(A);
    for (unsigned int chunk = blockIdx.x; chunk < A.n_chunks; chunk += gridDim.x) {
        if (A.chunk_count[chunk] == 0u) continue;   // uniform across the block
        const uint64_t lo = (uint64_t)chunk * kCmpChunk;
        if (tid == 0) s_run = A.chunk_pre[chunk];
        uint4 r[kCmpTiles];
#pragma unroll
        for (int t = 0; t < kCmpTiles; t++) {
            const uint64_t e = lo + (uint64_t)t * kCmpTile + (uint64_t)tid * 16;
            r[t] = e < A.count ? cmp_reason16(A, cls, e) : make_uint4(~0u, ~0u, ~0u, ~0u);
        }
        __syncthreads();
#pragma unroll
        for (int t = 0; t < kCmpTiles; t++) {
            const uint64_t e = lo + (uint64_t)t * kCmpTile + (uint64_t)tid * 16;
            uint32_t m = cmp_feasible16(r[t]);
            const unsigned int mine = (unsigned int)__popc(m);
            if (!__syncthreads_or((int)mine)) continue;
            unsigned int x = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned int y = __shfl_up_sync(0xFFFFFFFFu, x, off);
                if (lane >= off) x += y;
            }
            if (lane == 31) s_warp[warp] = x;
            __syncthreads();
            unsigned int before = 0, total = 0;
#pragma unroll
            for (int w = 0; w < kCmpThreads / 32; w++) {
                const unsigned int wt = s_warp[w];
                if (w < warp) before += wt;
                total += wt;
            }
            unsigned long long pos = s_run + before + (x - mine);
            const uint32_t w4[4] = {r[t].x, r[t].y, r[t].z, r[t].w};
            while (m) {
                const int i = __ffs(m) - 1;
                m &= m - 1;
                if (pos < A.record_cap) {
                    const uint64_t rel = e + i;
                    pf_record_t rec;
                    rec.idx = A.first + rel;
                    rec.mem = A.mem ? A.mem[rel] : 0;
                    rec.tput = A.tput[rel];
                    rec.reason = (uint8_t)((w4[i >> 2] >> (8 * (i & 3))) & 0xFFu);
                    rec.pad[0] = rec.pad[1] = rec.pad[2] = 0;
                    A.records[pos] = rec;
                }
                pos++;
            }
            __syncthreads();
            if (tid == 0) s_run += total;
            __syncthreads();
        }
        __syncthreads();
    }
}

// The feasibility bits of the chunks that hold a feasible plan, written to `mask` -- which may be page-locked HOST
// memory mapped into the device's address space: every other chunk's bits are zero and reach the host as one early
// copy of zeros instead of crossing the bus behind the search.  Runs after compact_count_kernel (chunk counts).
__global__ void __launch_bounds__(kCmpThreads) compact_mask_kernel(const CompactArgs A)
{
    const int tid = threadIdx.x;
    const uint8_t *cls = cmp_guard_cls(A);
    for (unsigned int chunk = blockIdx.x; chunk < A.n_chunks; chunk += gridDim.x) {
        if (A.chunk_count[chunk] == 0u) continue;   // uniform across the block
        const uint64_t lo = (uint64_t)chunk * kCmpChunk;
#pragma unroll
        for (int t = 0; t < kCmpTiles; t++) {
            const uint64_t e = lo + (uint64_t)t * kCmpTile + (uint64_t)tid * 16;
            const uint32_t m = e < A.count ? cmp_feasible16(cmp_reason16(A, cls, e)) : 0u;
            // two neighbours share one 32-bit store (e / 8 is a multiple of 4 in even threads); a pair that reaches
            // past the end of the range stores its bytes one by one
            const uint32_t up = __shfl_down_sync(0xFFFFFFFFu, m, 1);
            const uint64_t e_pair = e - (uint64_t)(tid & 1) * 16;
            if (e_pair + 32 <= A.count) {
                if ((tid & 1) == 0) *reinterpret_cast<uint32_t *>(A.mask + (e >> 3)) = m | (up << 16);
            } else if (e < A.count) {
                uint8_t *dst = A.mask + (e >> 3);
                dst[0] = (uint8_t)(m & 0xFFu);
                if (e + 8 < A.count) dst[1] = (uint8_t)(m >> 8);
            }
        }
    }
}

struct CompactLayout {
    size_t off_count, off_pre, total;
    unsigned int n_chunks;
};
static CompactLayout compact_layout(uint64_t count)
{
    CompactLayout l;
    l.n_chunks = (unsigned int)((count + kCmpChunk - 1) / kCmpChunk);
    if (l.n_chunks < 1) l.n_chunks = 1;
    l.off_count = 0;
    l.off_pre = ((size_t)l.n_chunks * 4 + 255) & ~(size_t)255;
    l.total = l.off_pre + (((size_t)l.n_chunks * 8 + 255) & ~(size_t)255);
    return l;
}

// The three launches on `st`.  guard: the class bytes of a scoring call whose constant blocks may still be in flight
// (NULL: the dense outputs are complete).  Arguments are the caller's to check.
int compact_run(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
                const int64_t *d_mem, uint64_t *d_hist, uint8_t *d_mask, pf_record_t *d_records, uint64_t record_cap,
                uint64_t *d_n_feasible, void *d_workspace, cudaStream_t st, const FillGuard *guard)
{
    const CompactLayout lay = compact_layout(count);
    uint8_t *ws = (uint8_t *)d_workspace;
    CompactArgs a;
    a.first = first; a.count = count; a.reason = d_reason; a.tput = d_tput; a.mem = (const long long *)d_mem;
    a.hist = (unsigned long long *)d_hist; a.mask = d_mask; a.records = record_cap ? d_records : nullptr;
    a.record_cap = record_cap; a.n_feasible = (unsigned long long *)d_n_feasible;
    a.chunk_count = (unsigned int *)(ws + lay.off_count);
    a.chunk_pre = (unsigned long long *)(ws + lay.off_pre);
    a.n_chunks = lay.n_chunks;
    if (guard) a.guard = *guard;
    PF_CUDA_TRY(cudaMemsetAsync(d_hist, 0, PF_REASON_BINS * sizeof(uint64_t), st), "pf_compact: histogram reset");
    timing_begin(p, PF_T_COMPACT, st);
    compact_count_kernel<<<lay.n_chunks, kCmpThreads, 0, st>>>(a);
    compact_scan_kernel<<<1, 1024, 0, st>>>(a);
    int launches = 2;
    if (record_cap > 0) {
        const unsigned int grid = lay.n_chunks < (unsigned int)p->sm_count * 8 ? lay.n_chunks : (unsigned int)p->sm_count * 8;
        compact_write_kernel<<<grid, kCmpThreads, 0, st>>>(a);
        launches++;
    }
    timing_end(p, PF_T_COMPACT, launches, st);
    for (int i = 0; i < launches; i++) count_launch();
    PF_CUDA_TRY(cudaGetLastError(), "pf_compact launch");
    return PF_OK;
}

// The bits of the chunks with feasible plans, after compact_run on the same stream and workspace (see
// compact_mask_kernel); `mask` is a device-visible address.
int compact_mask_run(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason, uint8_t *mask,
                     void *d_workspace, cudaStream_t st, const FillGuard *guard)
{
    const CompactLayout lay = compact_layout(count);
    uint8_t *ws = (uint8_t *)d_workspace;
    CompactArgs a = {};
    a.first = first; a.count = count; a.reason = d_reason; a.mask = mask;
    a.chunk_count = (unsigned int *)(ws + lay.off_count);
    a.chunk_pre = (unsigned long long *)(ws + lay.off_pre);
    a.n_chunks = lay.n_chunks;
    if (guard) a.guard = *guard;
    const unsigned int grid = lay.n_chunks < (unsigned int)p->sm_count * 8 ? lay.n_chunks : (unsigned int)p->sm_count * 8;
    compact_mask_kernel<<<grid, kCmpThreads, 0, st>>>(a);
    count_launch();
    PF_CUDA_TRY(cudaGetLastError(), "compact_mask_kernel launch");
    return PF_OK;
}

}  // namespace pf

using namespace pf;

extern "C" size_t pf_compact_workspace(uint64_t count)
{
    return compact_layout(count ? count : 1).total;
}

extern "C" int pf_compact(pf_plan_t *p, uint64_t first, uint64_t count, const uint8_t *d_reason, const float *d_tput,
                          const int64_t *d_mem, uint64_t *d_hist, uint8_t *d_mask, pf_record_t *d_records,
                          uint64_t record_cap, uint64_t *d_n_feasible, void *d_workspace, size_t workspace_bytes,
                          void *stream)
{
    if (!p || !d_reason || !d_hist || !d_n_feasible) return PF_EINVAL;
    if (record_cap > 0 && (!d_records || !d_tput)) return PF_EINVAL;
    if (count == 0 || count >= PF_MAX_COUNT) return PF_ERANGE;
    if (first >= p->size || count > p->size - first) return PF_ERANGE;
    const CompactLayout lay = compact_layout(count);
    if (!d_workspace || ((uintptr_t)d_workspace & 255) != 0 || workspace_bytes < lay.total) return PF_EWORKSPACE;
    if (int rc_dev = check_device(p)) return rc_dev;
    return compact_run(p, first, count, d_reason, d_tput, d_mem, d_hist, d_mask, d_records, record_cap, d_n_feasible,
                       d_workspace, (cudaStream_t)stream, nullptr);
}
