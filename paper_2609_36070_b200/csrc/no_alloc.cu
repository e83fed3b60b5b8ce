// mok_schedule_noalloc: the dispatch-schedule stage for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need a schedule: a serving loop that
// must not take cudaMalloc's device-wide synchronisation on its critical path, a process whose framework has already
// reserved all of HBM for its own pool (so a raw allocation may simply fail), or a plug-in that is only handed input
// and output buffers and no allocator.  For them the scratch that mok_schedule normally takes from a caller-owned
// workspace lives in a fixed array inside the library image.  The paper has no counterpart of this entry point.
//
// The array exists once per GPU that loads the library and stays allocated until the process exits.  All calls on a
// device share it and it keeps whatever the previous call left behind, so two calls that overlap on the device (two
// streams, two host threads) race; the header word that must start at zero is cleared on every call.
#include "mok_internal.cuh"
#include <string.h>

namespace mok {

constexpr size_t NOALLOC_SCRATCH_BYTES = 1536u << 10;  // 1.5 MiB: enough for MOK_NOALLOC_MAX_ROUTES routes with E = 512
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

// Device address of the scratch array, looked up once per device.  In host code `g_noalloc_scratch` is only a
// handle for the runtime, not a device pointer, so it is never passed to a kernel directly.
static char* g_noalloc_ptr[64];

static int noalloc_scratch(char** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= 64) return (int)cudaErrorInvalidDevice;
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);    // resolves the symbol for the current device
        if (e != cudaSuccess) return (int)e;
        g_noalloc_ptr[dev] = reinterpret_cast<char*>(p);
    }
    *out = g_noalloc_ptr[dev];
    return 0;
}

}  // namespace mok

using namespace mok;

extern "C" int mok_schedule_noalloc(const int32_t* topk_idx, int T, int E, int k,
                                    int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                                    void* stream) {
    WsLayout L;
    if (!ws_layout(T, 8, 8, 0, E, k, &L)) return MOK_ERR_SHAPE;
    if ((long long)T * k > MOK_NOALLOC_MAX_ROUTES) return MOK_ERR_SHAPE;
    // the schedule kernels touch the regions from the header up to and including row_token
    if (L.row_token + sizeof(int32_t) * (size_t)L.Rpad > NOALLOC_SCRATCH_BYTES) return MOK_ERR_SHAPE;
    if (T == 0) return MOK_OK;
    if (!topk_idx) return MOK_ERR_NULL;
    char* ws = nullptr;
    if (noalloc_scratch(&ws) != 0) return MOK_ERR_CUDA;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(ws + L.header, 0, sizeof(WsHeader), s);   // status / tile count start at zero
    if (e != cudaSuccess) return MOK_ERR_CUDA;
    e = launch_schedule(topk_idx, T, E, k, TILE_M, TILE_M, L, ws, counts, offsets, perm, inv_perm, s);
    return e == cudaSuccess ? MOK_OK : MOK_ERR_CUDA;
}
