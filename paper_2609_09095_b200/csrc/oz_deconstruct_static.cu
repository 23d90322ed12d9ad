// oz_deconstruct_static: the deconstruction stage for callers that cannot allocate device memory.
//
// Some callers of this library run where cudaMalloc is off limits: inside a framework whose
// caching allocator owns every byte and forbids raw allocations, in a real-time loop where an
// allocation's implicit synchronisation is unacceptable, or in a process whose memory budget was
// fixed before it started.  oz_deconstruct needs a small scratch area for its per-line scan
// results; this entry point keeps that scratch in a fixed array inside the library image, so the
// caller passes only the operand and the outputs.
//
// The array is one file-scope object per device (every GPU that loads the library holds it until
// the process exits).  In host code its name is only a stand-in: the device address is obtained
// with cudaGetSymbolAddress, once per device, with that device current, on the first call made
// on that device.  That first call should therefore come before any stream capture begins.
#include <mutex>

#include "oz_internal.h"

constexpr int64_t kStaticMaxLines = OZ_STATIC_MAX_LINES;
constexpr size_t kStaticScratchBytes = 16 * static_cast<size_t>(kStaticMaxLines) + 256;

// The scratch itself: 4 MiB + 256 bytes per device, zero-initialised at load, reused by every call.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_addr[kMaxDevices] = {};

// device address of the scratch array on the current device (looked up once per device)
oz_status_t static_scratch_address(void **out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return OZ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
        void *ptr = nullptr;
        cudaError_t rc = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_scratch);
        if (rc != cudaSuccess || !ptr) return OZ_ERR_CUDA;
        g_static_addr[dev] = ptr;
    }
    *out = g_static_addr[dev];
    return OZ_OK;
}

}  // namespace

extern "C" oz_status_t oz_deconstruct_static(int side, int64_t lines, int64_t k, const double *X,
                                             int64_t ldx, oz_modset_t set, uint32_t route,
                                             uint8_t *planes, int64_t plane_stride,
                                             int64_t row_pitch, int32_t *shift, void *stream)
{
    oz::Route rt;
    if ((set != OZ_SET_S && set != OZ_SET_E && set != OZ_SET_A) || !oz::decode_route_for_set(set, route, &rt) ||
        (side != 0 && side != 1))
        return OZ_ERR_INVALID_ARG;
    if (lines < 0 || k < 0) return OZ_ERR_INVALID_ARG;
    if (k > OZ_K_MAX) return OZ_ERR_UNSUPPORTED;
    if (oz::resolve_schedule(set, k, 0, false, &rt) != OZ_OK) return OZ_ERR_UNSUPPORTED;
    if (lines > kStaticMaxLines) return OZ_ERR_WORKSPACE;   // beyond the built-in scratch
    if (lines == 0) return OZ_OK;
    if (!planes || !shift || (k > 0 && !X)) return OZ_ERR_INVALID_ARG;
    if (row_pitch < k || row_pitch < 16 || (row_pitch & 15) || (plane_stride & 15) ||
        plane_stride < lines * row_pitch || (reinterpret_cast<uintptr_t>(planes) & 15u) ||
        (reinterpret_cast<uintptr_t>(shift) & 3u) || (reinterpret_cast<uintptr_t>(X) & 7u))
        return OZ_ERR_INVALID_ARG;
    if (k > 0 && ldx < (side == 0 ? lines : k)) return OZ_ERR_INVALID_ARG;
    oz_status_t st = oz::ensure_device_ready();
    if (st != OZ_OK) return st;
    void *scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != OZ_OK) return st;
    // The scan kernels clear the part of the scratch they use before accumulating into it, so the
    // previous call's contents never leak into this one.
    return oz::launch_deconstruct(side, lines, k, X, ldx, set, rt, planes, plane_stride, row_pitch,
                                  shift, scratch, static_cast<cudaStream_t>(stream));
}
