// gs_sample_batch_noalloc: the mini-batch call for hosts that must not allocate device memory.
//
// Some callers of this library run where cudaMalloc is off limits: a training loop whose memory
// was carved up front by a pool allocator that owns every byte of the device, a plugin that is
// handed buffers by its host application and may not grow the process' footprint, or a service
// with a fixed memory budget that is audited at start-up.  gs_sample_batch asks such a caller for
// a scratch workspace it has no way to provide.  This variant keeps the scratch inside the
// library instead, in a file-scope device array of fixed size; the caller passes only inputs and
// outputs.  The CUDA runtime materialises that array on a GPU the first time its address is
// looked up there, which gs_cache_init does (prepare_noalloc_scratch below), so the memory is
// taken at set-up, not in the middle of training, and is held until the process exits.
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

// Called by gs_cache_init / gs_cache_init_split with the cache's device current: looks the address
// up early, so that the array exists before the first batch and before any stream capture.
gs_status prepare_noalloc_scratch() {
    void* unused = nullptr;
    return scratch_address(&unused);
}

static bool is_aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

}  // namespace gs

using namespace gs;

extern "C" gs_status gs_sample_batch_noalloc(gs_cache* cache, const int32_t* d_seeds, int32_t num_seeds, gs_mode mode,
                                             double gamma, uint32_t step, int32_t* d_input_nodes,
                                             int64_t input_nodes_capacity, const gs_block_buffers* h_buffers,
                                             void* stream, gs_block* blocks, const int32_t** d_num_input_nodes) {
    if (!cache) return set_error(GS_ERR_ARG, "cache is NULL");
    if (!h_buffers) return set_error(GS_ERR_ARG, "h_buffers is NULL");
    if (!blocks) return set_error(GS_ERR_ARG, "blocks is NULL");
    // The relabel kernel stores block-local ids four at a time: 16-byte stores into d_indices.
    // Inside a workspace those arrays start on 256-byte boundaries; here they are the caller's, so
    // the requirement is checked before anything is launched.
    if (!is_aligned(d_input_nodes, 4)) return set_error(GS_ERR_ALIGN, "d_input_nodes must be 4-byte aligned");
    const int32_t hops = cache_num_hops(cache);
    for (int l = 0; l < hops; ++l) {
        if (!is_aligned(h_buffers[l].d_indptr, 4))
            return set_error(GS_ERR_ALIGN, "h_buffers[%d].d_indptr must be 4-byte aligned", l);
        if (!is_aligned(h_buffers[l].d_indices, 16))
            return set_error(GS_ERR_ALIGN, "h_buffers[%d].d_indices must be 16-byte aligned", l);
    }
    size_t need = 0;
    gs_status st = cache_workspace_bytes(cache, num_seeds, &need);
    if (st != GS_OK) return st;
    if (need > (size_t)GS_NOALLOC_SCRATCH_BYTES)
        return set_error(GS_ERR_WORKSPACE, "gs_sample_batch_noalloc: this batch needs %zu bytes of scratch, the built-in scratch "
                         "array has %u", need, (unsigned)GS_NOALLOC_SCRATCH_BYTES);
    void* scratch = nullptr;
    st = scratch_address(&scratch);
    if (st != GS_OK) return st;
    OutputBuffers out{};
    out.input_nodes = d_input_nodes;
    out.input_nodes_capacity = input_nodes_capacity;
    // the number of hops is private to the cache; the checked call below reads exactly that many entries
    for (int l = 0; l < GS_MAX_HOPS; ++l) {
        out.indptr[l] = nullptr;
        out.indices[l] = nullptr;
    }
    for (int l = 0; l < hops; ++l) {
        out.indptr[l] = h_buffers[l].d_indptr;
        out.indptr_capacity[l] = h_buffers[l].indptr_capacity;
        out.indices[l] = h_buffers[l].d_indices;
        out.indices_capacity[l] = h_buffers[l].indices_capacity;
    }
    const int32_t* d_in = nullptr;
    // Output buffers that are too small fail in here with GS_ERR_WORKSPACE, before any launch.
    return sample_batch_checked(cache, d_seeds, num_seeds, mode, gamma, step, scratch, (size_t)GS_NOALLOC_SCRATCH_BYTES,
                                (cudaStream_t)stream, blocks, &d_in, d_num_input_nodes, &out);
}
