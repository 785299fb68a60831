// pf_probe.cu -- micro-kernels that measure the denominators of the two rooflines the scoring path is held
// against: thread-instruction issue rate (independent FFMA, IMAD and LOP3/IADD chains at full occupancy)
// and the rate of a pure streaming write.  Measurement utilities only: the paper has no counterpart and no
// scoring call depends on them.  The caller times the launches with events on the stream it passes.
// Built into a library of its own (libplanfront_probe.so) and self-contained: nothing of the scoring library is
// linked in.
#include <cuda_runtime.h>
#include <stdint.h>

#include "planfront_bench.h"

#define PF_PROBE_TRY(expr)                       \
    do {                                         \
        if ((expr) != cudaSuccess) return PF_ECUDA; \
    } while (0)

namespace pf {

constexpr int kProbeThreads = 256;
constexpr int kProbeBlocksPerSM = 8;   // 2048 resident threads per SM
constexpr int kProbeChains = 8;        // independent dependency chains per thread
constexpr int kProbeUnroll = 4;        // chain steps per loop iteration

// Every chain step is one PTX instruction of the measured kind, written as volatile inline assembly so the
// compiler can neither fold nor reorder the chains; the loop counter and branch add 2 instructions per
// kProbeChains * kProbeUnroll measured ones and are not counted.
template <int KIND>
__global__ void __launch_bounds__(kProbeThreads) probe_alu_kernel(uint32_t iters, uint32_t seed, uint32_t *sink)
{
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x;
    if (KIND == PF_PROBE_FFMA) {
        float a[kProbeChains];
        const float x = 1.0f + 1e-7f * (float)(seed & 7), y = 1e-9f * (float)(tid & 15);
#pragma unroll
        for (int c = 0; c < kProbeChains; c++) a[c] = (float)(tid + c);
        for (uint32_t i = 0; i < iters; i++) {
#pragma unroll
            for (int u = 0; u < kProbeUnroll; u++)
#pragma unroll
                for (int c = 0; c < kProbeChains; c++)
                    asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(a[c]) : "f"(x), "f"(y));
        }
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < kProbeChains; c++) s += a[c];
        if (s == 12345.678f) sink[0] = tid;  // keeps the chains live; practically never taken
    } else {
        uint32_t a[kProbeChains];
        const uint32_t x = seed | 1u, y = tid * 2654435761u;
#pragma unroll
        for (int c = 0; c < kProbeChains; c++) a[c] = tid + (uint32_t)c;
        for (uint32_t i = 0; i < iters; i++) {
#pragma unroll
            for (int u = 0; u < kProbeUnroll; u++)
#pragma unroll
                for (int c = 0; c < kProbeChains; c++) {
                    if (KIND == PF_PROBE_IMAD)
                        asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(a[c]) : "r"(x), "r"(y));
                    else if ((c + u) & 1)
                        asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(a[c]) : "r"(x), "r"(y));
                    else
                        asm volatile("add.u32 %0, %0, %1;" : "+r"(a[c]) : "r"(y));
                }
        }
        uint32_t s = 0;
#pragma unroll
        for (int c = 0; c < kProbeChains; c++) s ^= a[c];
        if (s == 0x9e3779b9u && iters == 0xFFFFFFFFu) sink[0] = s;
    }
}

// 16-byte streaming stores, one per thread over a grid as large as the buffer: the fastest pure write on this
// part (a persistent grid-stride loop reaches about 0.82 of it, ticketed 156 KB chunks 0.96)
__global__ void __launch_bounds__(kProbeThreads) probe_write_kernel(uint4 *dst, uint64_t n16, uint32_t tag)
{
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n16) __stcs(dst + i, make_uint4(tag, tag, tag, tag));
}

static int sm_count(int *out)
{
    int dev = 0;
    PF_PROBE_TRY(cudaGetDevice(&dev));
    PF_PROBE_TRY(cudaDeviceGetAttribute(out, cudaDevAttrMultiProcessorCount, dev));
    return PF_OK;
}

}  // namespace pf

extern "C" int pf_probe_alu(int kind, uint32_t iters, uint32_t *d_sink, uint64_t *h_thread_instructions,
                            void *stream)
{
    using namespace pf;
    if (!d_sink || !h_thread_instructions || iters == 0 || iters > (1u << 24)) return PF_EINVAL;
    if (kind != PF_PROBE_FFMA && kind != PF_PROBE_IMAD && kind != PF_PROBE_LOGIC) return PF_EINVAL;
    int sms = 0;
    int rc = sm_count(&sms);
    if (rc != PF_OK) return rc;
    const int grid = sms * kProbeBlocksPerSM;
    cudaStream_t st = (cudaStream_t)stream;
    if (kind == PF_PROBE_FFMA)
        probe_alu_kernel<PF_PROBE_FFMA><<<grid, kProbeThreads, 0, st>>>(iters, 3u, d_sink);
    else if (kind == PF_PROBE_IMAD)
        probe_alu_kernel<PF_PROBE_IMAD><<<grid, kProbeThreads, 0, st>>>(iters, 3u, d_sink);
    else
        probe_alu_kernel<PF_PROBE_LOGIC><<<grid, kProbeThreads, 0, st>>>(iters, 3u, d_sink);
    PF_PROBE_TRY(cudaGetLastError());
    *h_thread_instructions = (uint64_t)grid * kProbeThreads * (uint64_t)iters * kProbeChains * kProbeUnroll;
    return PF_OK;
}

extern "C" int pf_probe_write(void *d_buf, size_t bytes, void *stream)
{
    using namespace pf;
    if (!d_buf || bytes < 16 || ((uintptr_t)d_buf & 15) != 0 || (bytes & 15) != 0) return PF_EINVAL;
    const uint64_t n16 = (uint64_t)(bytes / 16);
    const uint64_t blocks = (n16 + kProbeThreads - 1) / kProbeThreads;
    if (blocks > 0x7FFFFFFFull) return PF_EINVAL;
    probe_write_kernel<<<(unsigned int)blocks, kProbeThreads, 0, (cudaStream_t)stream>>>((uint4 *)d_buf, n16,
                                                                                        0x5a5a5a5au);
    PF_PROBE_TRY(cudaGetLastError());
    return PF_OK;
}
