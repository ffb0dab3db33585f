// Host-side helpers shared by the launchers: the driver's tensor-map encoder, the SM count of the
// current device, the once-per-device shared-memory opt-in of a kernel, and whether kernels are launched
// with programmatic dependent launch.
#include "common.cuh"
#include "tc_common.cuh"

#include <mutex>
#include <vector>

namespace npas {

// Multiprocessors of the current device (looked up once per device index).
int sm_count()
{
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cached[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    cached[dev].store(n, std::memory_order_relaxed);
    return n;
}

// Opt a kernel in to `bytes` of dynamic shared memory.  The attribute belongs to the (kernel, device) pair and
// stays set, so the runtime is asked only when a pair is new or wants more than it was given before.
npas_status allow_dynamic_smem(const void *kernel, int bytes)
{
    struct Entry { const void *kernel; int dev, bytes; };
    static std::mutex mu;
    static std::vector<Entry> seen;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NPAS_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    for (Entry &e : seen)
        if (e.kernel == kernel && e.dev == dev) {
            if (e.bytes >= bytes) return NPAS_OK;
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return NPAS_ERR_CUDA;
            e.bytes = bytes;
            return NPAS_OK;
        }
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return NPAS_ERR_CUDA;
    seen.push_back({kernel, dev, bytes});
    return NPAS_OK;
}

namespace tc {

bool pdl_enabled() { return true; }

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

}  // namespace tc
}  // namespace npas
