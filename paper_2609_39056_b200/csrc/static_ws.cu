// rudder_linear_static: rudder_linear for callers that cannot allocate device memory.
//
// The activation codes Q_X and the row scales r that pass between the two kernels normally live in
// a workspace the caller allocates.  Some callers have no allocator to ask: code running inside a
// framework's captured region or a real-time control loop where cudaMalloc is forbidden, plug-ins
// that are handed input and output tensors only, or hosts whose memory pool is owned by someone
// else.  For them the scratch lives here, in a fixed array inside the library image.
#include "internal.cuh"

namespace {

// Every GPU that loads the library holds this array until the process exits.
constexpr size_t kStaticWorkspaceBytes = size_t(4) << 20;   // 4 MiB
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

// In host code `g_static_workspace` is only a handle for the symbol, not a device address: the
// address the kernels may use has to be asked for, once per device, with that device current.
void* g_static_workspace_addr[64] = {nullptr};

rudder_status static_workspace(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return RUDDER_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_state_mutex);
    if (g_static_workspace_addr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || ptr == nullptr) return RUDDER_ERR_CUDA;
        g_static_workspace_addr[dev] = ptr;
    }
    *out = g_static_workspace_addr[dev];
    return RUDDER_OK;
}

}  // namespace

extern "C" {

size_t rudder_linear_static_max_workspace_bytes(void) { return kStaticWorkspaceBytes; }

rudder_status rudder_linear_static(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M,
                                   const rudder_segments* seg, int step, const rudder_scale_table* tab,
                                   const float* bias, uint16_t* Y, int64_t ldy, void* stream)
{
    if (!w) return RUDDER_ERR_ARG;
    if (M < 1) return RUDDER_ERR_SHAPE;
    // Too large for the fixed array: refuse before anything is launched.
    if (workspace_bytes_for(w, M) > kStaticWorkspaceBytes) return RUDDER_ERR_WORKSPACE;
    void* ws = nullptr;
    rudder_status s = static_workspace(&ws);
    if (s != RUDDER_OK) return s;
    // Nothing has to be cleared: the prologue overwrites every code and row scale the GEMM reads, and
    // rows past M are zero-filled by the TMA bounds, not read from the array.
    return linear_impl(w, X, ldx, M, seg, step, tab, bias, Y, ldy, ws, kStaticWorkspaceBytes,
                       static_cast<cudaStream_t>(stream), nullptr, 0, 0, 0, 0);
}

}  // extern "C"
