// npas_conv2d_bp_static_ws: the block-punched convolution for callers that cannot hand the
// library any device scratch of their own.  The kernels' device status words live in a small
// file-scope array that every GPU loading this library carries until the process exits.
#include "common.cuh"

#include <mutex>

namespace {

constexpr size_t kStaticWsBytes = 256;   // the whole scratch need of one call, whatever its shape
static_assert(kStaticWsBytes >= NPAS_WORKSPACE_BYTES, "static scratch smaller than a call's need");

// Device-resident scratch.  In host code this name is only a handle for the runtime's symbol
// lookup, never an address a kernel may be given: the real device address is fetched once per
// device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_ws_addr[kMaxDevices] = {};

// Device address of g_static_ws on the current device (looked up on the first call per device).
npas_status static_ws_address(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NPAS_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ws_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) return NPAS_ERR_CUDA;
        g_ws_addr[dev] = p;
    }
    *out = g_ws_addr[dev];
    return NPAS_OK;
}

}  // namespace

extern "C" npas_status npas_conv2d_bp_static_ws(const npas_conv_desc *d, const npas_bp_desc *bp,
                                                const void *x_dev, const void *blob_dev,
                                                const float *bias_dev, const void *residual_dev,
                                                void *y_dev, int32_t *device_status_host, void *stream)
{
    if (NPAS_WORKSPACE_BYTES > kStaticWsBytes) return NPAS_ERR_BUFFER_TOO_SMALL;
    // arguments first: nothing is enqueued for a call that will be refused
    int32_t kernel_id = 0;
    npas_status s = npas_conv2d_bp_kernel(d, bp, &kernel_id);
    if (s != NPAS_OK) return s;
    if (!x_dev || !blob_dev || !y_dev) return NPAS_ERR_NULL;
    size_t need = 0;
    s = npas_conv2d_bp_workspace(d, bp, &need);
    if (s != NPAS_OK) return s;
    if (need > kStaticWsBytes) return NPAS_ERR_BUFFER_TOO_SMALL;
    void *ws = nullptr;
    s = static_ws_address(&ws);
    if (s != NPAS_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: start this call from clean status words
    if (cudaMemsetAsync(ws, 0, kStaticWsBytes, st) != cudaSuccess) return NPAS_ERR_CUDA;
    s = npas_conv2d_bp(d, bp, x_dev, blob_dev, bias_dev, residual_dev, y_dev, ws, kStaticWsBytes, stream);
    if (s != NPAS_OK || !device_status_host) return s;
    uint32_t w[2] = {0, 0};
    if (cudaMemcpyAsync(w, ws, sizeof w, cudaMemcpyDeviceToHost, st) != cudaSuccess) return NPAS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return NPAS_ERR_CUDA;
    *device_status_host = (int32_t)w[0];
    if (w[0] == 0) return NPAS_OK;
    return w[0] == (uint32_t)NPAS_ERR_BLOB ? NPAS_ERR_BLOB : NPAS_ERR_TIMEOUT;
}
