// rago_search_probes_noalloc: the coarse step (query-to-centroid scores + nprobe selection) for
// callers that cannot provide or allocate scratch memory.  The score matrix, which rago_search_probes
// keeps in the caller's workspace, lives here in a fixed array that is part of the library image.
#include <mutex>

#include "plan.cuh"

namespace rago {

// Scratch of the no-allocation entry point.  The array is part of the library image: a GPU holds these bytes
// from the moment the runtime loads this module on it until the process exits.  The runtime loads modules on
// first use, so that moment is the first look-up of the array's address on the device, which rago_index_load
// does (noalloc_prepare below): the memory is claimed, and a failure reported, when an index is loaded, not
// in the middle of serving.
static __device__ __align__(256) unsigned char g_static_scratch[RAGO_NOALLOC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
static std::mutex g_setup_mutex;
static void* g_scratch_ptr[MAX_DEVICES];  // device address of g_static_scratch, per device ordinal

// Device address of the array on the current device.  In host code `g_static_scratch` is only a
// handle for the runtime, so the address has to be asked for (once per device, that device current).
static cudaError_t scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

// Called by rago_index_load with the index's device current: resolves (and thereby makes resident) the array.
cudaError_t noalloc_prepare() {
    void* p = nullptr;
    return scratch_address(&p);
}

}  // namespace rago

using namespace rago;

extern "C" rago_status rago_search_probes_noalloc(const rago_index* index, const float* queries, int32_t nq,
                                                  int32_t nprobe, int32_t* out_lists, float* out_coarse,
                                                  void* cuda_stream) {
    const IndexImpl* ix = reinterpret_cast<const IndexImpl*>(index);
    if (!ix) { set_error("index is null"); return RAGO_EINVAL; }
    if (nq < 0) { set_error("nq = %d is negative", nq); return RAGO_EINVAL; }
    if (nprobe < 1 || nprobe > ix->nlist) {
        set_error("nprobe = %d outside [1, nlist = %d]", nprobe, ix->nlist);
        return RAGO_EINVAL;
    }
    if (nprobe > MAX_K) { set_error("nprobe = %d exceeds %d", nprobe, MAX_K); return RAGO_EUNSUPPORTED; }
    if (ix->tree_n1) { set_error("this entry point scores every list: not available while a two-level quantiser is set"); return RAGO_EUNSUPPORTED; }
    if (nq == 0) return RAGO_OK;
    if (!queries || !out_lists || !out_coarse) { set_error("null pointer"); return RAGO_EINVAL; }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != ix->device) {  // the array's address is per device
        set_error("the current device (%d) is not the index's device (%d)", dev, ix->device);
        return RAGO_EINVAL;
    }
    if (reinterpret_cast<uintptr_t>(queries) % 16) { set_error("queries need 16-byte alignment"); return RAGO_EALIGN; }
    // layout inside the fixed array: [scores nq*nlist f32][bias nq*nprobe f32], each 256-byte aligned
    const size_t scores_bytes = align_up((size_t)nq * ix->nlist * 4, 256);
    const size_t bias_bytes = align_up((size_t)nq * nprobe * 4, 256);
    const size_t need = scores_bytes + bias_bytes;
    if (need > (size_t)RAGO_NOALLOC_SCRATCH_BYTES) {
        set_error("batch too large for the built-in scratch: nq * nlist = %lld scores need %zu bytes, the limit is %d "
                  "(split the batch, or use rago_search_probes with a workspace)",
                  (long long)nq * ix->nlist, need, (int)RAGO_NOALLOC_SCRATCH_BYTES);
        return RAGO_ENOMEM;
    }
    void* base = nullptr;  // cached since rago_index_load; the look-up below only runs if that one failed
    cudaError_t e = scratch_address(&base);
    if (e != cudaSuccess) { set_error("cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e)); return RAGO_ECUDA; }
    float* scores = reinterpret_cast<float*>(base);
    float* bias = reinterpret_cast<float*>(static_cast<unsigned char*>(base) + scores_bytes);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // Nothing in the array has to start at zero: the first kernel writes every score the second one
    // reads, and the bias block is write-only here.
    e = launch_coarse_scores(ix, queries, nq, scores, nullptr, s);
    if (e == cudaSuccess)
        e = launch_select_probes(ix, queries, scores, nq, nprobe, out_lists, out_coarse, bias, nullptr, s);
    if (e != cudaSuccess) { set_error("coarse kernels: %s", cudaGetErrorString(e)); return RAGO_ECUDA; }
    return RAGO_OK;
}
