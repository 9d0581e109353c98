// GCN aggregation for callers that cannot supply (or allocate) a workspace: the per-segment partial
// sums of hub rows live in a fixed array inside the library image instead of a caller buffer.
#include <mutex>

#include "common.cuh"

namespace gnnfd {

constexpr size_t kStaticScratchBytes = GNNFD_STATIC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Lives in every device that loads the library, for the life of the process.  Host code must not use
// this name as an address: it is only a handle for cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

static std::mutex g_static_mutex;
static void* g_static_ptr[kMaxDevices];          // device address of g_static_scratch, per device ordinal

// Device address of the array on the current device; resolved on the first call per device.
static int static_scratch_address(void** out)
{
    int device = -1;
    GNNFD_CUDA_CHECK(cudaGetDevice(&device));
    if (device < 0 || device >= kMaxDevices) return GNNFD_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        GNNFD_CUDA_CHECK(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return GNNFD_CUDA_ERROR;
        g_static_ptr[device] = p;
    }
    *out = g_static_ptr[device];
    return GNNFD_OK;
}

}  // namespace gnnfd

extern "C" int gnnfd_aggregate_gcn_static(const gnnfd_csr_t* csr, const void* d_x, int64_t ldx, gnnfd_dtype_t xdt,
                                          void* d_out, int64_t ldo, gnnfd_dtype_t odt, int32_t f, int32_t chunk_width,
                                          void* stream)
{
    using namespace gnnfd;
    if (!csr || f <= 0) return GNNFD_INVALID_ARG;
    size_t need = 0;
    int rc = gnnfd_aggregate_workspace_bytes(csr, f, &need);
    if (rc) return rc;
    if (need > kStaticScratchBytes) return GNNFD_STATIC_SCRATCH_EXCEEDED;
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc) return rc;
    // Every partial sum that the reduction reads is written by the gather kernel of the same call, so
    // nothing in the array has to be cleared between calls.
    return gnnfd_aggregate_gcn(csr, d_x, ldx, xdt, d_out, ldo, odt, f, chunk_width, scratch, kStaticScratchBytes, stream);
}
