// gdn_tree_verify_static: tree verification for callers that must not allocate device memory.
//
// gdn_tree_verify needs device scratch (per-node tree metadata and the solve result of the general kernel) and
// asks its caller to provide it.  Some callers of this library have no way to get such a buffer:
// a serving process that handed all free device memory to its own pool at start-up and would see
// cudaMalloc fail, a decode loop in which cudaMalloc's implicit device-wide synchronisation would
// stall every other stream, or a plug-in living under a host whose memory policy forbids
// allocations by plug-ins.  For them the scratch lives here, in a fixed array that is part of the
// library image: every GPU that loads the library holds GDN_STATIC_SCRATCH_BYTES of it until the
// process exits, and nothing is ever allocated or freed.
#include <mutex>

#include "gdn_internal.cuh"

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime's symbol table,
// not a device address: it must go through cudaGetSymbolAddress before a kernel can be given it.
static __device__ __align__(256) unsigned char g_static_scratch[GDN_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// Device address of the scratch array on the current device (resolved once per device).
int scratch_for_current_device(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GDN_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return GDN_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return GDN_OK;
}

}  // namespace

extern "C" int gdn_tree_verify_static(const gdn_shape_t *shape, const float *S0, const void *q,
                                      const void *k, const void *v, const void *g, const void *beta,
                                      const int32_t *parent, const int32_t *node_offsets, void *o,
                                      int32_t *status_dev, void *cuda_stream)
{
    const size_t need = gdn_tree_workspace_bytes(shape);
    if (need == 0)   // invalid shape: let the ordinary entry point name the reason (it launches nothing)
        return gdn_tree_verify(shape, S0, q, k, v, g, beta, parent, node_offsets, o, nullptr, 0, status_dev,
                               cuda_stream);
    if (need > GDN_STATIC_SCRATCH_BYTES) return GDN_ERR_WORKSPACE;   // problem too large for the fixed scratch
    void *scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != GDN_OK) return rc;
    return gdn_tree_verify(shape, S0, q, k, v, g, beta, parent, node_offsets, o, scratch,
                           GDN_STATIC_SCRATCH_BYTES, status_dev, cuda_stream);
}
