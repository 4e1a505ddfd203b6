// gs_sample_batch_noalloc: the mini-batch call for hosts that must not allocate device memory.
//
// Some callers of this library run where cudaMalloc is off limits: a training loop whose memory
// was carved up front by a pool allocator that owns every byte of the device, a plugin that is
// handed buffers by its host application and may not grow the process' footprint, or a service
// with a fixed memory budget that is audited at start-up.  gs_sample_batch asks such a caller for
// a scratch workspace it has no way to provide.  This variant keeps the scratch inside the
// library instead, in a file-scope device array of fixed size that every GPU using the library
// holds from load to exit; the caller passes only inputs and outputs.
#include <cstdio>
#include <mutex>

#include "gs_internal.h"

namespace gs {

// The scratch itself.  In host code this name is only a stand-in for the symbol - it is NOT a
// device address and must never be handed to a kernel; the address is looked up per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[GS_NOALLOC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
static void* g_scratch_ptr[MAX_DEVICES];   // device address of the array on each GPU (NULL = not looked up yet)
static std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device; looked up once per device.
static gs_status scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return set_error(GS_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= MAX_DEVICES) return set_error(GS_ERR_ARG, "device ordinal %d not supported", dev);
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p)
            return set_error(GS_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return GS_OK;
}

}  // namespace gs

using namespace gs;

extern "C" gs_status gs_sample_batch_noalloc(gs_cache* cache, const int32_t* d_seeds, int32_t num_seeds, gs_mode mode,
                                             double gamma, uint32_t step, int32_t* d_input_nodes,
                                             int64_t input_nodes_capacity, const gs_block_buffers* h_buffers,
                                             void* stream, gs_block* blocks, const int32_t** d_num_input_nodes) {
    if (!cache) return set_error(GS_ERR_ARG, "cache is NULL");
    if (!h_buffers) return set_error(GS_ERR_ARG, "h_buffers is NULL");
    if (!blocks) return set_error(GS_ERR_ARG, "blocks is NULL");
    void* scratch = nullptr;
    gs_status st = scratch_address(&scratch);
    if (st != GS_OK) return st;
    OutputBuffers out{};
    out.input_nodes = d_input_nodes;
    out.input_nodes_capacity = input_nodes_capacity;
    // the number of hops is private to the cache; the checked call below reads exactly that many entries
    for (int l = 0; l < GS_MAX_HOPS; ++l) {
        out.indptr[l] = nullptr;
        out.indices[l] = nullptr;
    }
    const int32_t hops = cache_num_hops(cache);
    for (int l = 0; l < hops; ++l) {
        out.indptr[l] = h_buffers[l].d_indptr;
        out.indptr_capacity[l] = h_buffers[l].indptr_capacity;
        out.indices[l] = h_buffers[l].d_indices;
        out.indices_capacity[l] = h_buffers[l].indices_capacity;
    }
    const int32_t* d_in = nullptr;
    // A batch whose scratch does not fit the array fails here with GS_ERR_WORKSPACE and a message
    // that names both sizes; nothing is launched in that case.
    st = sample_batch_checked(cache, d_seeds, num_seeds, mode, gamma, step, scratch, (size_t)GS_NOALLOC_SCRATCH_BYTES,
                              (cudaStream_t)stream, blocks, &d_in, d_num_input_nodes, &out);
    if (st == GS_ERR_WORKSPACE) {
        // keep the message of the size check, but say which buffer it is about
        char msg[400];
        snprintf(msg, sizeof(msg), "%s", gs_last_error());
        return set_error(GS_ERR_WORKSPACE, "gs_sample_batch_noalloc (built-in scratch of %u bytes): %s",
                         (unsigned)GS_NOALLOC_SCRATCH_BYTES, msg);
    }
    return st;
}
