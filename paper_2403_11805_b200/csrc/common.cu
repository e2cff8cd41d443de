// Status strings, CUDA error capture, descriptor checks and record-size arithmetic (host only).
#include <stdio.h>
#include <string.h>

#include "llms_internal.cuh"

namespace llms {

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e, const char *where)
{
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
    cudaGetLastError();  // clear a non-sticky error so that the next call starts clean
}

int sm_count()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

void *device_view_of_pinned(const void *host_ptr)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host_ptr) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer)
        return attr.devicePointer;
    cudaGetLastError();
    return nullptr;
}

int check_desc(const llms_kv_desc *d)
{
    if (!d) return LLMS_ERR_INVALID_ARG;
    if (d->n_layers <= 0 || d->n_kv_heads <= 0 || d->n_q_heads <= 0 || d->head_dim <= 0) return LLMS_ERR_INVALID_ARG;
    if (d->n_tokens <= 0 || d->chunk_len <= 0) return LLMS_ERR_INVALID_ARG;
    if (d->n_q_heads % d->n_kv_heads) return LLMS_ERR_INVALID_ARG;
    if (d->stride_l < 0 || d->stride_s < 0 || d->stride_h < 0) return LLMS_ERR_INVALID_ARG;
    if (d->quant_mode == 0) {
        if (d->group_size <= 0 || d->head_dim % d->group_size) return LLMS_ERR_INVALID_ARG;
    } else if (d->quant_mode != 1) {
        return LLMS_ERR_INVALID_ARG;
    }
    return LLMS_OK;
}

int check_desc_codec(const llms_kv_desc *d)
{
    int rc = check_desc(d);
    if (rc) return rc;
    if (d->head_dim % 16) return LLMS_ERR_MISALIGNED;
    if ((d->stride_l | d->stride_s | d->stride_h) % 8) return LLMS_ERR_MISALIGNED;
    if (d->quant_mode == 0) {
        if (!is_pow2(d->group_size) || d->group_size < 16 || d->group_size > 512) return LLMS_ERR_UNSUPPORTED;
    }
    return LLMS_OK;
}

}  // namespace llms

using namespace llms;

extern "C" const char *llms_strerror(int status)
{
    switch (status) {
    case LLMS_OK: return "ok";
    case LLMS_ERR_INVALID_ARG: return "invalid argument";
    case LLMS_ERR_BAD_BITS: return "bit-width must be 1, 2, 4 or 8";
    case LLMS_ERR_MISALIGNED: return "pointer, stride or offset is not aligned as required";
    case LLMS_ERR_BUF_TOO_SMALL: return "buffer or workspace too small";
    case LLMS_ERR_CUDA: return "CUDA runtime error";
    case LLMS_ERR_TIMEOUT: return "timed out";
    case LLMS_ERR_CORRUPT: return "record checksum mismatch";
    case LLMS_ERR_UNSUPPORTED: return "not supported by the kernels";
    default: return "unknown status";
    }
}

extern "C" const char *llms_last_cuda_error(void) { return g_cuda_error; }

extern "C" int llms_record_layout(const llms_kv_desc *desc, int bits, uint64_t *codes_offset, uint64_t *nbytes)
{
    int rc = check_desc(desc);
    if (rc) return rc;
    rc = check_bits(bits);
    if (rc) return rc;
    const uint64_t n_elem = (uint64_t)slabs_per_chunk(*desc) * (uint64_t)slab_elems(*desc);
    if ((n_elem * (uint64_t)bits) % 8) return LLMS_ERR_INVALID_ARG;
    const uint64_t co = round_up(groups_per_chunk(*desc) * 4, 16);
    if (codes_offset) *codes_offset = co;
    if (nbytes) *nbytes = round_up(co + n_elem * (uint64_t)bits / 8, 256);
    return LLMS_OK;
}

extern "C" int llms_record_bytes(const llms_kv_desc *desc, int bits, uint64_t *nbytes)
{
    return llms_record_layout(desc, bits, nullptr, nbytes);
}

extern "C" int llms_compressed_size(const llms_kv_desc *desc, const uint8_t *bits, int n, uint64_t *nbytes)
{
    if (n < 0 || (n > 0 && !bits) || !nbytes) return LLMS_ERR_INVALID_ARG;
    uint64_t total = 0;
    for (int i = 0; i < n; ++i) {
        uint64_t nb;
        int rc = llms_record_bytes(desc, bits[i], &nb);
        if (rc) return rc;
        total += nb;
    }
    *nbytes = total;
    return LLMS_OK;
}

extern "C" int llms_codec_workspace_bytes(int n, uint64_t *nbytes)
{
    if (n < 0 || !nbytes) return LLMS_ERR_INVALID_ARG;
    *nbytes = ws_total(n);
    return LLMS_OK;
}
