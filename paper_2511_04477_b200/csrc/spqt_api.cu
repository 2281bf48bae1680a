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

// ---------------------------------------------------------------- host-buffer path

// x from pinned host memory into its device staging buffer by a kernel (one CTA): for the few KB of a hidden
// state the copy engine's start-up latency is several times the transfer, while a kernel's loads over the bus
// take one round trip when they are all in flight together.  16-byte loads when both sides allow it.
constexpr int kFetchMax = 8;   // vectors per launch of the fetch kernel
struct FetchList {
    const unsigned short* src[kFetchMax];
    unsigned short* dst[kFetchMax];
    int n[kFetchMax];
};

__global__ void __launch_bounds__(256) fetch_x_kernel(FetchList fl)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned short* __restrict__ src = fl.src[blockIdx.x];
    unsigned short* __restrict__ dst = fl.dst[blockIdx.x];
    const int n = fl.n[blockIdx.x];
    const int tid = threadIdx.x;
    if (((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) == 0) {
        const int nv = n >> 3;   // whole 16-byte pieces
        const uint4* s4 = reinterpret_cast<const uint4*>(src);
        uint4* d4 = reinterpret_cast<uint4*>(dst);
        for (int i0 = 0; i0 < nv; i0 += 256 * 8) {
            uint4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = i0 + j * 256 + tid;
                if (i < nv) v[j] = s4[i];
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = i0 + j * 256 + tid;
                if (i < nv) d4[i] = v[j];
            }
        }
        for (int i = (nv << 3) + tid; i < n; i += 256) dst[i] = src[i];
    } else {
        for (int i = tid; i < n; i += 256) dst[i] = src[i];
    }
}

// the device address of pinned host memory the device can reach, or nullptr
static void* device_view(const void* host_ptr)
{
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host_ptr) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer != nullptr)
        return attr.devicePointer;
    (void)cudaGetLastError();  // pageable memory is not an error here
    return nullptr;
}

static spqt_status launch_fetch(const FetchList& fl, int count, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(count);
    cfg.blockDim = dim3(256);
    cfg.stream = s;
    cudaLaunchAttribute la[1];
    la[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    la[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = la;
    cfg.numAttrs = g_no_pdl ? 0 : 1;
    if (cudaLaunchKernelEx(&cfg, fetch_x_kernel, fl) != cudaSuccess) return SPQT_ERR_CUDA;
    count_launch();
    return SPQT_OK;
}

static spqt_status linear_host(const void* codes, const void* scale_zero, int m, int n, int bits, int group,
                               const void* x_host, float t, void* y_host,
                               void* x_dev, int32_t* idx_dev, int32_t* count_dev, void* y_dev,
                               void* workspace, size_t workspace_bytes, void* stream, bool wait, bool x_in_place = false)
{
    if (!x_host || !y_host || !x_dev || !y_dev) return SPQT_ERR_INVALID_ARG;
    Format f;
    spqt_status st = make_format(m, n, bits, group, &f);
    if (st != SPQT_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // x: fetched by a small kernel if x_host is pinned memory the device can address, by a copy otherwise
    // (x_in_place: the caller has already brought it to x_dev)
    if (!x_in_place) {
        if (void* xv = device_view(x_host)) {
            FetchList fl = {};
            fl.src[0] = static_cast<const unsigned short*>(xv);
            fl.dst[0] = static_cast<unsigned short*>(x_dev);
            fl.n[0] = n;
            if (launch_fetch(fl, 1, s) != SPQT_OK) return SPQT_ERR_CUDA;
        } else if (cudaMemcpyAsync(x_dev, x_host, (size_t)n * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) {
            return SPQT_ERR_CUDA;
        }
    }
    // If y_host is pinned memory the device can address, the kernel writes y there itself (posted
    // writes over the bus) and the copy back, with its start-up latency, is not needed.
    void* y_target = y_dev;
    if (void* yv = device_view(y_host)) y_target = yv;
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

struct HostStep {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
};

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

spqt_status spqt_sparse_linear_host(const void* codes, const void* scale_zero,
                                    int m, int n, int bits, int group,
                                    const void* x_host, float t, void* y_host,
                                    void* x_dev, int32_t* idx_dev, int32_t* count_dev, void* y_dev,
                                    void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::linear_host(codes, scale_zero, m, n, bits, group, x_host, t, y_host, x_dev, idx_dev, count_dev, y_dev,
                       workspace, workspace_bytes, stream, true);
}

spqt_status spqt_sparse_linear_host_async(const void* codes, const void* scale_zero,
                                          int m, int n, int bits, int group,
                                          const void* x_host, float t, void* y_host,
                                          void* x_dev, int32_t* idx_dev, int32_t* count_dev, void* y_dev,
                                          void* workspace, size_t workspace_bytes, void* stream)
{
    return spqt::linear_host(codes, scale_zero, m, n, bits, group, x_host, t, y_host, x_dev, idx_dev, count_dev, y_dev,
                       workspace, workspace_bytes, stream, false);
}


spqt_status spqt_host_step_create(const spqt_host_linear* linears, int count, void** step)
{
    if (!linears || count < 1 || !step) return SPQT_ERR_INVALID_ARG;
    *step = nullptr;
    cudaStream_t s = nullptr;
    if (cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess) return SPQT_ERR_CUDA;
    spqt_status st = SPQT_OK;
    spqt::HostStep* h = new spqt::HostStep();
    if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        st = SPQT_ERR_CUDA;
    } else {
        // every x the device can reach is fetched at the head of the step (one CTA per vector), so that the
        // linears then follow one another without a transfer in between
        bool* fetched = new bool[count]();
        spqt::FetchList fl = {};
        int k = 0;
        for (int i = 0; i < count && st == SPQT_OK; ++i) {
            const spqt_host_linear& l = linears[i];
            void* xv = (l.x_host && l.x_dev && l.n > 0) ? spqt::device_view(l.x_host) : nullptr;
            if (xv) {
                fl.src[k] = static_cast<const unsigned short*>(xv);
                fl.dst[k] = static_cast<unsigned short*>(l.x_dev);
                fl.n[k] = l.n;
                fetched[i] = true;
                ++k;
            }
            if (k == spqt::kFetchMax || (i == count - 1 && k > 0)) {
                st = spqt::launch_fetch(fl, k, s);
                k = 0;
            }
        }
        for (int i = 0; i < count && st == SPQT_OK; ++i) {
            const spqt_host_linear& l = linears[i];
            st = spqt::linear_host(l.codes, l.scale_zero, l.m, l.n, l.bits, l.group, l.x_host, l.t, l.y_host, l.x_dev, l.idx_dev,
                             l.count_dev, l.y_dev, l.workspace, l.workspace_bytes, s, false, fetched[i]);
        }
        delete[] fetched;
        if (cudaStreamEndCapture(s, &h->graph) != cudaSuccess || h->graph == nullptr) {
            if (st == SPQT_OK) st = SPQT_ERR_CUDA;
        }
        if (st == SPQT_OK && cudaGraphInstantiate(&h->exec, h->graph, 0) != cudaSuccess) st = SPQT_ERR_CUDA;
    }
    (void)cudaStreamDestroy(s);
    if (st != SPQT_OK) {
        (void)cudaGetLastError();
        if (h->exec) (void)cudaGraphExecDestroy(h->exec);
        if (h->graph) (void)cudaGraphDestroy(h->graph);
        delete h;
        return st;
    }
    *step = h;
    return SPQT_OK;
}

spqt_status spqt_host_step_launch(void* step, void* stream)
{
    if (!step) return SPQT_ERR_INVALID_ARG;
    spqt::HostStep* h = static_cast<spqt::HostStep*>(step);
    return cudaGraphLaunch(h->exec, static_cast<cudaStream_t>(stream)) == cudaSuccess ? SPQT_OK : SPQT_ERR_CUDA;
}

spqt_status spqt_host_step_destroy(void* step)
{
    if (!step) return SPQT_ERR_INVALID_ARG;
    spqt::HostStep* h = static_cast<spqt::HostStep*>(step);
    (void)cudaGraphExecDestroy(h->exec);
    (void)cudaGraphDestroy(h->graph);
    delete h;
    return SPQT_OK;
}

}  // extern "C"
