// A plain streaming kernel with the codec's access shape (every load or store instruction of a warp covers 1 KiB of
// consecutive bytes in 256-bit accesses) and a chosen mix of bytes read to bytes written.  It does nothing useful: it
// measures what the memory system gives such a stream, which is the yardstick the codec kernels' throughput is read
// against (the encoder reads about four bytes for each one it writes, the decoder the reverse).
//
// Work split of the yardstick: one warp per iteration and then the warp is done, eight consecutive iterations per CTA,
// CTAs handed to the SMs in address order by the hardware as earlier ones leave: of the splits tried this one gives
// the most.  Two more splits can be asked for, to see what a split costs: resident CTAs whose warps stride through the
// buffer (the memory system does not serve all SMs at the same rate, and a fixed split waits for the slowest), and
// resident CTAs whose warps draw their iterations from counters, which is what the codec kernels do.
#include <algorithm>

#include "llms_internal.cuh"

namespace llms {

constexpr int kProbeThreads = 256;
constexpr int kProbeCounters = 16, kProbeCounterStride = 32;   // words; as in the codec kernels
__device__ uint32_t g_probe_counters[kProbeCounters * kProbeCounterStride];

template <int RK>
__device__ __forceinline__ void probe_load(const uint8_t *__restrict__ src, uint64_t i, int lane, uint32_t (&w)[RK > 0 ? RK : 1][8])
{
#pragma unroll
    for (int k = 0; k < RK; ++k) {
        const uint8_t *p = src + (i * RK + k) * 1024 + lane * 32;
        asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(w[k][0]), "=r"(w[k][1]), "=r"(w[k][2]), "=r"(w[k][3]), "=r"(w[k][4]), "=r"(w[k][5]), "=r"(w[k][6]),
                       "=r"(w[k][7])
                     : "l"(p));
    }
}

template <int RK, int WK>
__device__ __forceinline__ void probe_store(uint8_t *__restrict__ dst, uint64_t i, int lane, const uint32_t (&w)[RK > 0 ? RK : 1][8],
                                            uint32_t &acc)
{
#pragma unroll
    for (int k = 0; k < RK; ++k)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc ^= w[k][j];
#pragma unroll
    for (int k = 0; k < WK; ++k) {
        uint8_t *p = dst + (i * WK + k) * 1024 + lane * 32;
        const uint32_t v = (uint32_t)i;
        asm volatile("st.global.L1::no_allocate.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                     :: "r"(v), "r"(v), "r"(v), "r"(v), "r"(v), "r"(v), "r"(v), "r"(v), "l"(p) : "memory");
    }
}

// DRAWN = false: warp w takes iterations w, w + W, w + 2W, ...  With a grid of one warp per iteration that is one
// iteration per warp (the yardstick); with a grid of resident CTAs it is the fixed split the codec kernels had once.
// DRAWN = true (resident CTAs): the codec kernels' split - a warp's first batch of two iterations is its own number,
// every further batch number is drawn, one draw ahead of need, from one of 16 counters (zero at the launch).
template <int RK, int WK, bool DRAWN>
__global__ void __launch_bounds__(kProbeThreads) stream_probe_kernel(const uint8_t *__restrict__ src, uint8_t *__restrict__ dst,
                                                                     uint64_t iters, uint32_t *sink)
{
    const int lane = threadIdx.x & 31;
    const uint64_t n_warps = (uint64_t)gridDim.x * (kProbeThreads / 32);
    const uint64_t gw = (uint64_t)blockIdx.x * (kProbeThreads / 32) + (threadIdx.x >> 5);
    uint32_t acc = 0;
    uint32_t wa[RK > 0 ? RK : 1][8], wb[RK > 0 ? RK : 1][8];
    if constexpr (!DRAWN) {
        for (uint64_t i = gw; i < iters; i += n_warps) {
            probe_load<RK>(src, i, lane, wa);
            probe_store<RK, WK>(dst, i, lane, wa, acc);
        }
    } else {
        const uint32_t slot = (uint32_t)(gw % kProbeCounters);
        uint32_t *ctr = g_probe_counters + slot * kProbeCounterStride;
        uint64_t base = gw * 2;
        while (base < iters) {
            uint32_t drawn = 0;
            if (lane == 0) drawn = atomicAdd(ctr, 1u);
            const bool two = base + 1 < iters;
            probe_load<RK>(src, base, lane, wa);         // the loads of the whole batch are in flight together
            if (two) probe_load<RK>(src, base + 1, lane, wb);
            probe_store<RK, WK>(dst, base, lane, wa, acc);
            if (two) probe_store<RK, WK>(dst, base + 1, lane, wb, acc);
            drawn = __shfl_sync(0xffffffffu, drawn, 0);
            base = (n_warps + (uint64_t)drawn * kProbeCounters + slot) * 2;
        }
    }
    if (acc == 0x9E3779B9u && sink) *sink = acc;   // keeps the loads alive; practically never taken
}

}  // namespace llms

using namespace llms;

extern "C" int llms_stream_probe_split(const void *src, uint64_t src_bytes, void *dst, uint64_t dst_bytes, uint64_t iters,
                                       int read_kib, int write_kib, int split, void *stream)
{
    if (iters == 0 || read_kib < 0 || write_kib < 0 || read_kib + write_kib == 0) return LLMS_ERR_INVALID_ARG;
    if (split < 0 || split > 2) return LLMS_ERR_INVALID_ARG;
    if ((read_kib > 0 && !src) || (write_kib > 0 && !dst)) return LLMS_ERR_INVALID_ARG;
    if (!aligned(src, 32) || !aligned(dst, 32)) return LLMS_ERR_MISALIGNED;
    if (iters > (1ull << 40) || iters * (uint64_t)read_kib * 1024 > src_bytes || iters * (uint64_t)write_kib * 1024 > dst_bytes)
        return LLMS_ERR_BUF_TOO_SMALL;
    const uint64_t want = (iters + kProbeThreads / 32 - 1) / (kProbeThreads / 32);
    // split 0: a warp per iteration (in practice); 1 and 2: resident CTAs, two per SM like the codec kernels
    const int grid = (int)std::min<uint64_t>(want, split == 0 ? 0x7fffffffull : (uint64_t)sm_count() * 2);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint8_t *s = static_cast<const uint8_t *>(src);
    uint8_t *d = static_cast<uint8_t *>(dst);
    if (split == 2) {
        void *counters = nullptr;
        LLMS_CUDA_TRY(cudaGetSymbolAddress(&counters, g_probe_counters));
        LLMS_CUDA_TRY(cudaMemsetAsync(counters, 0, sizeof(uint32_t) * kProbeCounters * kProbeCounterStride, st));
    }
#define LLMS_PROBE(R, W)                                                                                  \
    if (read_kib == R && write_kib == W) {                                                                \
        if (split == 2) stream_probe_kernel<R, W, true><<<grid, kProbeThreads, 0, st>>>(s, d, iters, nullptr);  \
        else stream_probe_kernel<R, W, false><<<grid, kProbeThreads, 0, st>>>(s, d, iters, nullptr);      \
        LLMS_CUDA_TRY(cudaGetLastError());                                                                \
        return LLMS_OK;                                                                                   \
    }
    LLMS_PROBE(4, 0)
    LLMS_PROBE(0, 4)
    LLMS_PROBE(4, 1)
    LLMS_PROBE(1, 4)
    LLMS_PROBE(2, 2)
#undef LLMS_PROBE
    return LLMS_ERR_UNSUPPORTED;
}

extern "C" int llms_stream_probe(const void *src, uint64_t src_bytes, void *dst, uint64_t dst_bytes, uint64_t iters,
                                 int read_kib, int write_kib, void *stream)
{
    return llms_stream_probe_split(src, src_bytes, dst, dst_bytes, iters, read_kib, write_kib, 0, stream);
}
