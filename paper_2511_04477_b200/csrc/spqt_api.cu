// Entry points that launch nothing themselves: status names, buffer sizes,
// tuning knobs, device queries, and the host-buffer convenience call.
#include <atomic>

#include "spqt_common.cuh"

namespace spqt {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int k) { g_launches.fetch_add((unsigned long long)k, std::memory_order_relaxed); }

int sm_count()
{
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
        cached[dev] = v;
    }
    return cached[dev];
}

}  // namespace spqt

extern "C" {

const char* spqt_status_string(int s)
{
    switch (s) {
        case SPQT_OK: return "SPQT_OK";
        case SPQT_ERR_INVALID_ARG: return "SPQT_ERR_INVALID_ARG";
        case SPQT_ERR_UNSUPPORTED: return "SPQT_ERR_UNSUPPORTED";
        case SPQT_ERR_ALIGNMENT: return "SPQT_ERR_ALIGNMENT";
        case SPQT_ERR_WORKSPACE: return "SPQT_ERR_WORKSPACE";
        case SPQT_ERR_CUDA: return "SPQT_ERR_CUDA";
        case SPQT_ERR_TIMEOUT: return "SPQT_ERR_TIMEOUT";
        default: return "SPQT_ERR_UNKNOWN";
    }
}

int spqt_version(void) { return 2000; }

spqt_status spqt_packed_sizes(int m, int n, int bits, int group,
                              size_t* codes_bytes, size_t* scale_zero_bytes,
                              size_t* gemv_workspace_bytes)
{
    spqt::Format f;
    spqt_status st = spqt::make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    if (codes_bytes) *codes_bytes = f.blocks * (size_t)f.B;
    if (scale_zero_bytes) *scale_zero_bytes = f.blocks * 4;
    if (gemv_workspace_bytes) *gemv_workspace_bytes = spqt::workspace_bytes(f);
    return SPQT_OK;
}

unsigned long long spqt_launch_count(void) { return spqt::g_launches.load(std::memory_order_relaxed); }

static spqt_status linear_host(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                               const void* x_host, float t, void* y_host,
                               void* x_dev, int32_t* idx_dev, int32_t* count_dev, void* y_dev,
                               void* workspace, size_t workspace_bytes, void* stream, bool wait)
{
    if (!x_host || !y_host || !x_dev || !y_dev) return SPQT_ERR_INVALID_ARG;
    spqt::Format f;
    spqt_status st = spqt::make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(x_dev, x_host, (size_t)n * 2, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return SPQT_ERR_CUDA;
    // If y_host is pinned memory the device can address, the kernel writes y there itself (posted
    // writes over the bus) and the copy back, with its start-up latency, is not needed.
    void* y_target = y_dev;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, y_host) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
        attr.devicePointer != nullptr)
        y_target = attr.devicePointer;
    else
        (void)cudaGetLastError();  // pageable memory is not an error here
    // index collection and product in one launch (two for very long x: the call decides)
    st = spqt_sparsify_gemv(codes, scale_zero, m, n, bits, group, x_dev, t, idx_dev, count_dev,
                            y_target, workspace, workspace_bytes, stream);
    if (st != SPQT_OK) return st;
    if (y_target == y_dev &&
        cudaMemcpyAsync(y_host, y_dev, (size_t)m * 2, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return SPQT_ERR_CUDA;
    if (wait && cudaStreamSynchronize(s) != cudaSuccess) return SPQT_ERR_CUDA;
    return SPQT_OK;
}

spqt_status spqt_sparse_linear_host(const void* codes, const void* scale_zero,
                                    int m, int n, int bits, int group,
                                    const void* x_host, float t, void* y_host,
                                    void* x_dev, int32_t* idx_dev, int32_t* count_dev, void* y_dev,
                                    void* workspace, size_t workspace_bytes, void* stream)
{
    return linear_host(codes, scale_zero, m, n, bits, group, x_host, t, y_host, x_dev, idx_dev, count_dev, y_dev,
                       workspace, workspace_bytes, stream, true);
}

spqt_status spqt_sparse_linear_host_async(const void* codes, const void* scale_zero,
                                          int m, int n, int bits, int group,
                                          const void* x_host, float t, void* y_host,
                                          void* x_dev, int32_t* idx_dev, int32_t* count_dev, void* y_dev,
                                          void* workspace, size_t workspace_bytes, void* stream)
{
    return linear_host(codes, scale_zero, m, n, bits, group, x_host, t, y_host, x_dev, idx_dev, count_dev, y_dev,
                       workspace, workspace_bytes, stream, false);
}

}  // extern "C"
