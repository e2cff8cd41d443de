// Swap copies: packed records between a device swap buffer and a pinned host arena on a side stream.
#include <chrono>
#include <thread>

#include "llms_internal.cuh"

namespace llms {

// Issue the copies of n records; runs adjacent on both sides are merged into one cudaMemcpyAsync.
static int copy_records(uint8_t *dst, const uint8_t *src, const llms_chunk_meta *meta, const uint64_t *host_offsets,
                        int n, bool to_host, cudaStream_t st)
{
    int i = 0;
    while (i < n) {
        const uint64_t dev0 = meta[i].offset;
        const uint64_t host0 = host_offsets ? host_offsets[i] : meta[i].offset;
        uint64_t len = meta[i].nbytes;
        int j = i + 1;
        while (j < n) {
            const uint64_t hj = host_offsets ? host_offsets[j] : meta[j].offset;
            if (meta[j].offset != dev0 + len || hj != host0 + len) break;
            len += meta[j].nbytes;
            ++j;
        }
        if (to_host) LLMS_CUDA_TRY(cudaMemcpyAsync(dst + host0, src + dev0, len, cudaMemcpyDeviceToHost, st));
        else LLMS_CUDA_TRY(cudaMemcpyAsync(dst + dev0, src + host0, len, cudaMemcpyHostToDevice, st));
        i = j;
    }
    return LLMS_OK;
}

static int check_swap(const void *a, const void *b, const llms_chunk_meta *meta, const uint64_t *host_offsets, int n,
                      uint64_t dev_bytes, uint64_t host_bytes)
{
    if (n < 0) return LLMS_ERR_INVALID_ARG;
    if (n == 0) return LLMS_OK;
    if (!a || !b || !meta) return LLMS_ERR_INVALID_ARG;
    if (!aligned(a, 16) || !aligned(b, 16)) return LLMS_ERR_MISALIGNED;
    for (int i = 0; i < n; ++i) {
        if (meta[i].nbytes == 0 || meta[i].nbytes % 256 || meta[i].offset % 256) return LLMS_ERR_MISALIGNED;
        if (host_offsets && host_offsets[i] % 16) return LLMS_ERR_MISALIGNED;
    }
    // every record inside both buffers (written so that nothing can wrap around)
    for (int i = 0; i < n; ++i) {
        const uint64_t host_off = host_offsets ? host_offsets[i] : meta[i].offset;
        if (meta[i].nbytes > dev_bytes || meta[i].offset > dev_bytes - meta[i].nbytes) return LLMS_ERR_BUF_TOO_SMALL;
        if (meta[i].nbytes > host_bytes || host_off > host_bytes - meta[i].nbytes) return LLMS_ERR_BUF_TOO_SMALL;
    }
    return LLMS_OK;
}

}  // namespace llms

using namespace llms;

extern "C" int llms_swap_out(const void *dev_buf, uint64_t dev_bytes, const llms_chunk_meta *meta, int n, void *pinned_dst,
                             uint64_t host_bytes, const uint64_t *host_offsets, void *side_stream, void *after, void *done)
{
    int rc = check_swap(dev_buf, pinned_dst, meta, host_offsets, n, dev_bytes, host_bytes);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(side_stream);
    if (after) LLMS_CUDA_TRY(cudaStreamWaitEvent(st, static_cast<cudaEvent_t>(after), 0));
    rc = copy_records(static_cast<uint8_t *>(pinned_dst), static_cast<const uint8_t *>(dev_buf), meta, host_offsets, n, true, st);
    if (rc) return rc;
    if (done) LLMS_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(done), st));
    return LLMS_OK;
}

extern "C" int llms_swap_in(const void *pinned_src, uint64_t host_bytes, const uint64_t *host_offsets,
                            const llms_chunk_meta *meta, int n, void *dev_buf, uint64_t dev_bytes, void *side_stream,
                            void *after, void *done)
{
    int rc = check_swap(pinned_src, dev_buf, meta, host_offsets, n, dev_bytes, host_bytes);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(side_stream);
    if (after) LLMS_CUDA_TRY(cudaStreamWaitEvent(st, static_cast<cudaEvent_t>(after), 0));
    rc = copy_records(static_cast<uint8_t *>(dev_buf), static_cast<const uint8_t *>(pinned_src), meta, host_offsets, n, false, st);
    if (rc) return rc;
    if (done) LLMS_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(done), st));
    return LLMS_OK;
}

extern "C" int llms_wait(void *event, uint32_t timeout_ms)
{
    if (!event) return LLMS_ERR_INVALID_ARG;
    const auto start = std::chrono::steady_clock::now();
    const auto deadline = start + std::chrono::milliseconds(timeout_ms);
    const auto spin_until = start + std::chrono::microseconds(200);   // short waits are polled without giving the core up
    for (;;) {
        const cudaError_t e = cudaEventQuery(static_cast<cudaEvent_t>(event));
        if (e == cudaSuccess) return LLMS_OK;
        if (e != cudaErrorNotReady) {
            set_cuda_error(e, "cudaEventQuery");
            return LLMS_ERR_CUDA;
        }
        const auto now = std::chrono::steady_clock::now();
        if (now >= deadline) return LLMS_ERR_TIMEOUT;
        if (now >= spin_until) std::this_thread::sleep_for(std::chrono::microseconds(20));
    }
}
